// Host side of the library: tensor registry, trace store, roofline classifier and planner.
// Integer arithmetic only (128-bit products); no CUDA call in this file.
#include "tgp_internal.h"
#include <algorithm>
#include <cstring>
#include <deque>
#include <thread>

typedef unsigned __int128 u128;
static const uint64_t ALIGN = 512;      // placement granularity in the arena
static const int32_t W_AFF = 4;         // ops a tensor may sit unused and still keep its place
static const uint64_t ZC_DEN = 2;       // an access touching < size/ZC_DEN of a read-only tensor is served in place

static inline uint64_t alignup(uint64_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

int tgp_fail(tgp_ctx *ctx, int code, const std::string &msg) { if (ctx) ctx->err = msg; return code; }

template <class T> static void put(std::vector<uint8_t> &b, T v) {
    const uint8_t *p = (const uint8_t *)&v; b.insert(b.end(), p, p + sizeof(T));
}

static int give(const std::vector<uint8_t> &b, void *buf, uint64_t *bytes) {
    if (!bytes) return TGP_E_INVAL;
    if (buf) { if (*bytes < b.size()) return TGP_E_INVAL; memcpy(buf, b.data(), b.size()); }
    *bytes = b.size();
    return TGP_OK;
}

extern "C" {

const char *tgp_strerror(int code) {
    switch (code) {
    case TGP_OK: return "ok";
    case TGP_E_INVAL: return "invalid argument or call order";
    case TGP_E_OVERLAP: return "sub-range overlaps a registered tensor";
    case TGP_E_RANGE: return "address or sub-range outside the pool";
    case TGP_E_UNKNOWN_TENSOR: return "unknown tensor id";
    case TGP_E_BUDGET_TOO_SMALL: return "device budget too small for this trace";
    case TGP_E_NO_PLAN: return "no plan";
    case TGP_E_CUDA: return "CUDA call failed";
    case TGP_E_MISMATCH: return "run-time access differs from the trace";
    case TGP_E_STATE: return "wrong state for this call";
    case TGP_E_TOO_LARGE: return "size beyond the fixed maximum";
    default: return "unknown error code";
    }
}

const char *tgp_last_error(const tgp_ctx *ctx) { return ctx ? ctx->err.c_str() : ""; }

int tgp_create(tgp_ctx **out, const tgp_machine *m) {
    if (!out || !m || !m->peak_flops || !m->hbm_Bps || !m->h2d_Bps || !m->d2h_Bps) return TGP_E_INVAL;
    tgp_ctx *c = new (std::nothrow) tgp_ctx();
    if (!c) return TGP_E_INVAL;
    c->mach = *m;
    *out = c;
    return TGP_OK;
}

void tgp_destroy(tgp_ctx *ctx) {
    if (!ctx) return;
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();
    tgp_engine_free(ctx);
    delete ctx;
}

// ---- registry -------------------------------------------------------------------------------------
int tgp_pool_register(tgp_ctx *ctx, void *host_base, uint64_t bytes, uint32_t flags, uint32_t *pool_id) {
    if (!ctx || !host_base || !bytes || !pool_id) return TGP_E_INVAL;
    if ((uintptr_t)host_base % ALIGN) return tgp_fail(ctx, TGP_E_INVAL, "pool base not 512-byte aligned");
    uint32_t k = flags & (TGP_POOL_PINNED | TGP_POOL_MANAGED | TGP_POOL_PLAIN);
    if (k != TGP_POOL_PINNED && k != TGP_POOL_MANAGED && k != TGP_POOL_PLAIN)
        return tgp_fail(ctx, TGP_E_INVAL, "exactly one pool kind flag is required");
    for (auto &p : ctx->pools)
        if ((char *)host_base < p.host_base + p.bytes && p.host_base < (char *)host_base + bytes)
            return tgp_fail(ctx, TGP_E_OVERLAP, "pool overlaps a registered pool");
    ctx->pools.push_back({(char *)host_base, bytes, k, nullptr, false});
    *pool_id = (uint32_t)ctx->pools.size() - 1;
    return TGP_OK;
}

static void sort_by_addr(tgp_ctx *ctx) {
    if (!ctx->by_addr_dirty) return;
    std::sort(ctx->by_addr.begin(), ctx->by_addr.end(), [&](uint32_t a, uint32_t b) {
        const TgpTensor &x = ctx->tensors[a], &y = ctx->tensors[b];
        return x.pool != y.pool ? x.pool < y.pool : x.off < y.off;
    });
    ctx->by_addr_dirty = false;
}

// index in by_addr of the last tensor of `pool` starting at or before `off`, or -1
static long find_le(tgp_ctx *ctx, uint32_t pool, uint64_t off) {
    sort_by_addr(ctx);
    long lo = 0, hi = (long)ctx->by_addr.size();
    while (lo < hi) {
        long mid = (lo + hi) / 2;
        const TgpTensor &t = ctx->tensors[ctx->by_addr[mid]];
        if (t.pool < pool || (t.pool == pool && t.off <= off)) lo = mid + 1; else hi = mid;
    }
    return lo - 1;
}

int tgp_tensor_register(tgp_ctx *ctx, uint32_t pool, uint64_t offset, uint64_t bytes, uint64_t site_hash,
                        int32_t layer, uint32_t kind, uint32_t flags, uint32_t *tensor_id) {
    if (!ctx || !tensor_id || !bytes) return TGP_E_INVAL;
    if (pool >= ctx->pools.size()) return tgp_fail(ctx, TGP_E_INVAL, "unknown pool");
    if (flags != TGP_T_READONLY && flags != TGP_T_MUTABLE) return tgp_fail(ctx, TGP_E_INVAL, "tensor flags");
    if (offset % ALIGN) return tgp_fail(ctx, TGP_E_INVAL, "sub-range offset not 512-byte aligned");
    if (offset > ctx->pools[pool].bytes || bytes > ctx->pools[pool].bytes - offset)
        return tgp_fail(ctx, TGP_E_RANGE, "sub-range outside the pool");
    if (ctx->traced || ctx->tracing) return tgp_fail(ctx, TGP_E_STATE, "registry is frozen once tracing starts");
    long i = find_le(ctx, pool, offset);
    if (i >= 0) {
        const TgpTensor &p = ctx->tensors[ctx->by_addr[i]];
        if (p.pool == pool && p.off + p.size > offset) return tgp_fail(ctx, TGP_E_OVERLAP, "overlaps the tensor before it");
    }
    if (i + 1 < (long)ctx->by_addr.size()) {
        const TgpTensor &n = ctx->tensors[ctx->by_addr[i + 1]];
        if (n.pool == pool && n.off < offset + bytes) return tgp_fail(ctx, TGP_E_OVERLAP, "overlaps the tensor after it");
    }
    uint64_t cnt = ctx->site_counter[site_hash]++;
    ctx->tensors.push_back({pool, offset, bytes, site_hash, cnt, layer, kind, flags});
    uint32_t id = (uint32_t)ctx->tensors.size() - 1;
    // keep by_addr sorted cheaply when registrations come in address order (the usual case)
    if (!ctx->by_addr.empty()) {
        const TgpTensor &last = ctx->tensors[ctx->by_addr.back()];
        if (last.pool > pool || (last.pool == pool && last.off > offset)) ctx->by_addr_dirty = true;
    }
    ctx->by_addr.push_back(id);
    *tensor_id = id;
    return TGP_OK;
}

int tgp_tensor_lookup(const tgp_ctx *cctx, const void *host_addr, uint32_t *tensor_id, uint64_t *inner_offset) {
    tgp_ctx *ctx = const_cast<tgp_ctx *>(cctx);
    if (!ctx || !host_addr || !tensor_id) return TGP_E_INVAL;
    for (uint32_t p = 0; p < ctx->pools.size(); ++p) {
        const TgpPool &pl = ctx->pools[p];
        if ((const char *)host_addr < pl.host_base || (const char *)host_addr >= pl.host_base + pl.bytes) continue;
        uint64_t off = (uint64_t)((const char *)host_addr - pl.host_base);
        long i = find_le(ctx, p, off);
        if (i >= 0) {
            const TgpTensor &t = ctx->tensors[ctx->by_addr[i]];
            if (t.pool == p && off < t.off + t.size) {
                *tensor_id = ctx->by_addr[i];
                if (inner_offset) *inner_offset = off - t.off;
                return TGP_OK;
            }
        }
        return tgp_fail(ctx, TGP_E_RANGE, "address in a pool but in no registered sub-range");
    }
    return tgp_fail(ctx, TGP_E_RANGE, "address in no registered pool");
}

int tgp_tensor_identity(const tgp_ctx *ctx, uint32_t id, uint64_t *site_hash, uint64_t *counter) {
    if (!ctx || id >= ctx->tensors.size()) return TGP_E_UNKNOWN_TENSOR;
    if (site_hash) *site_hash = ctx->tensors[id].site_hash;
    if (counter) *counter = ctx->tensors[id].counter;
    return TGP_OK;
}

// ---- trace ----------------------------------------------------------------------------------------
int tgp_trace_begin(tgp_ctx *ctx) {
    if (!ctx) return TGP_E_INVAL;
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();
    ctx->tail_ready = false; ctx->base_plan = TgpPlan();
    ctx->ops.clear(); ctx->acc.clear(); ctx->steps.clear();
    ctx->measured_ns.clear();
    ctx->plan = TgpPlan();
    ctx->tracing = true; ctx->traced = false;
    return TGP_OK;
}

int tgp_trace_step(tgp_ctx *ctx, uint32_t step_kind) {
    if (!ctx || !ctx->tracing) return TGP_E_STATE;
    if (step_kind != TGP_PREFILL && step_kind != TGP_DECODE) return TGP_E_INVAL;
    ctx->steps.push_back({step_kind, (uint32_t)ctx->ops.size(), 0});
    return TGP_OK;
}

int tgp_trace_op(tgp_ctx *ctx, uint64_t op_site, int32_t layer, uint32_t op_kind, uint64_t flops,
                 uint64_t hbm_bytes, uint32_t n_acc, const tgp_access *acc) {
    if (!ctx || !ctx->tracing || ctx->steps.empty()) return TGP_E_STATE;
    if (n_acc && !acc) return TGP_E_INVAL;
    for (uint32_t k = 0; k < n_acc; ++k) {
        if (acc[k].tensor >= ctx->tensors.size()) return tgp_fail(ctx, TGP_E_UNKNOWN_TENSOR, "trace names an unregistered tensor");
        if (acc[k].mode < 1 || acc[k].mode > 3) return tgp_fail(ctx, TGP_E_INVAL, "access mode");
        if ((acc[k].mode & TGP_W) && ctx->tensors[acc[k].tensor].flags != TGP_T_MUTABLE)
            return tgp_fail(ctx, TGP_E_INVAL, "write access to a read-only tensor");
        for (uint32_t j = 0; j < k; ++j)
            if (acc[j].tensor == acc[k].tensor) return tgp_fail(ctx, TGP_E_INVAL, "tensor listed twice in one op");
    }
    ctx->ops.push_back({(uint32_t)ctx->steps.size() - 1, op_site, layer, op_kind, flops, hbm_bytes,
                        (uint32_t)ctx->acc.size(), n_acc});
    ctx->acc.insert(ctx->acc.end(), acc, acc + n_acc);
    ctx->steps.back().nops++;
    return TGP_OK;
}

int tgp_trace_end(tgp_ctx *ctx) {
    if (!ctx || !ctx->tracing) return TGP_E_STATE;
    ctx->tracing = false; ctx->traced = true;
    return TGP_OK;
}

int tgp_trace_export(const tgp_ctx *ctx, void *buf, uint64_t *bytes) {
    if (!ctx || !ctx->traced) return TGP_E_STATE;
    std::vector<uint8_t> b;
    b.reserve(ctx->ops.size() * 40 + ctx->acc.size() * 16);
    for (const TgpOp &o : ctx->ops) {
        put<uint32_t>(b, o.step); put<uint64_t>(b, o.site); put<int32_t>(b, o.layer); put<uint32_t>(b, o.kind);
        put<uint64_t>(b, o.flops); put<uint64_t>(b, o.hbm); put<uint32_t>(b, o.nacc);
        for (uint32_t k = 0; k < o.nacc; ++k) {
            const tgp_access &a = ctx->acc[o.acc0 + k];
            put<uint32_t>(b, a.tensor); put<uint32_t>(b, a.mode); put<uint64_t>(b, a.touched_bytes);
        }
    }
    return give(b, buf, bytes);
}

// ---- policy ---------------------------------------------------------------------------------------
int tgp_set_budget(tgp_ctx *ctx, uint64_t bytes) {
    if (!ctx || !bytes) return TGP_E_INVAL;
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();      // a re-plan under way reads these inputs
    ctx->tail_ready = false;
    ctx->budget = bytes; ctx->plan.valid = false;
    return TGP_OK;
}

int tgp_set_replan_keep(tgp_ctx *ctx, int keep) {
    if (!ctx) return TGP_E_INVAL;
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();
    ctx->replan_keep = keep != 0;
    return TGP_OK;
}

int tgp_set_measured_times(tgp_ctx *ctx, const uint64_t *op_ns, uint64_t n_ops) {
    if (!ctx) return TGP_E_INVAL;
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();      // a re-plan under way reads these inputs
    ctx->tail_ready = false;
    if (!n_ops) { ctx->measured_ns.clear(); ctx->plan.valid = false; return TGP_OK; }
    if (!op_ns) return TGP_E_INVAL;
    if (!ctx->traced || n_ops != ctx->ops.size()) return tgp_fail(ctx, TGP_E_STATE, "one time per op of the finished trace is required");
    ctx->measured_ns.assign(op_ns, op_ns + n_ops);
    ctx->plan.valid = false;
    return TGP_OK;
}

int tgp_set_variant(tgp_ctx *ctx, uint32_t variant, uint32_t bits) {
    if (!ctx || variant > TGP_VAR_MANAGED_OBJECT || (bits & ~15u)) return TGP_E_INVAL;
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();      // a re-plan under way reads these inputs
    ctx->tail_ready = false;
    ctx->variant = variant; ctx->bits = bits; ctx->plan.valid = false;
    return TGP_OK;
}

int tgp_set_object_bytes(tgp_ctx *ctx, uint64_t bytes) {
    if (!ctx || bytes < (64u << 10)) return TGP_E_INVAL;
    ctx->object_bytes = bytes;
    return TGP_OK;
}

static uint8_t classify(const tgp_machine &m, uint64_t flops, uint64_t hbm, uint64_t mig, bool selective, uint64_t measured_ns) {
    if (mig > 0 && !selective) return CLS_LINK;
    if (measured_ns > 0) {
        // runtime monitor: the measured kernel time replaces both analytic roofs in the link test, mig/Bl > t
        if ((u128)mig * 1000000000ull > (u128)measured_ns * m.h2d_Bps) return CLS_LINK;
        return (u128)flops * m.hbm_Bps >= (u128)hbm * m.peak_flops ? CLS_COMPUTE : CLS_HBM;
    }
    // link time strictly above both other roofs: mig/Bl > flops/P and mig/Bl > hbm/Bh
    if ((u128)mig * m.peak_flops > (u128)flops * m.h2d_Bps && (u128)mig * m.hbm_Bps > (u128)hbm * m.h2d_Bps) return CLS_LINK;
    if ((u128)flops * m.hbm_Bps >= (u128)hbm * m.peak_flops) return CLS_COMPUTE;
    return CLS_HBM;
}

}  // extern "C"

// Builds the plan for the steps from first_step on (0: the whole run) into `out`; op indices are those of the whole
// trace.  A tail plan starts from an empty arena with every tensor written in an earlier step holding data in the
// pool (its first access loads it, write or not).  Touches nothing of ctx but `out` and `err`, so it may run on a
// helper thread while tgp_step() executes the current plan.
static int build_plan(const tgp_ctx *ctx, uint32_t first_step, TgpPlan &out, std::string &err) {
    auto fail = [&](int code, const char *msg) { err = msg; return code; };
    const size_t T = ctx->tensors.size(), N = ctx->ops.size();
    const size_t O0 = ctx->steps[first_step].op0;
    const std::vector<TgpTensor> &ten = ctx->tensors;
    TgpPlan pl;
    pl.first_step = first_step; pl.first_op = (uint32_t)O0;
    pl.cls.resize(N); pl.crit.assign(T, 0); pl.zc.assign(T, 0); pl.score.assign(T, 0);
    // classes, criticality, score
    for (size_t i = O0; i < N; ++i) {
        const TgpOp &o = ctx->ops[i];
        uint64_t mig = 0;
        for (uint32_t k = 0; k < o.nacc; ++k) mig += ctx->acc[o.acc0 + k].touched_bytes;
        pl.cls[i] = classify(ctx->mach, o.flops, o.hbm, mig, ctx->bits & TGP_BIT_P, ctx->measured_ns.size() == N ? ctx->measured_ns[i] : 0);
        if (pl.cls[i] == CLS_LINK)
            for (uint32_t k = 0; k < o.nacc; ++k) {
                const tgp_access &a = ctx->acc[o.acc0 + k];
                // link bytes residency would save: what the op touches, plus the whole-tensor write-back a write causes
                pl.crit[a.tensor] = 1; pl.score[a.tensor] += a.touched_bytes + ((a.mode & TGP_W) ? ten[a.tensor].size : 0);
            }
    }
    // zero-copy: read-only, accessed, and every access sparse
    {
        std::vector<uint8_t> accessed(T, 0), sparse(T, 1);
        for (size_t q = ctx->ops[O0].acc0; q < ctx->acc.size(); ++q) {
            const tgp_access &a = ctx->acc[q];
            accessed[a.tensor] = 1;
            if ((u128)a.touched_bytes * ZC_DEN >= ten[a.tensor].size) sparse[a.tensor] = 0;
        }
        if (ctx->bits & TGP_BIT_ZC)
            for (size_t t = 0; t < T; ++t) pl.zc[t] = accessed[t] && sparse[t] && ten[t].flags == TGP_T_READONLY;
    }
    // stays: maximal runs of accesses of one tensor within a step with gaps <= W_AFF ops
    struct Stay { int32_t first, last; };
    std::vector<std::vector<Stay>> stays(T);
    {
        std::vector<int32_t> last_op(T, -1);
        for (size_t i = O0; i < N; ++i) {
            const TgpOp &o = ctx->ops[i];
            for (uint32_t k = 0; k < o.nacc; ++k) {
                uint32_t t = ctx->acc[o.acc0 + k].tensor;
                if (pl.zc[t]) continue;
                if (last_op[t] >= 0 && (int32_t)i <= last_op[t] + W_AFF && ctx->ops[last_op[t]].step == o.step)
                    stays[t].back().last = (int32_t)i;
                else
                    stays[t].push_back({(int32_t)i, (int32_t)i});
                last_op[t] = (int32_t)i;
            }
        }
    }
    uint64_t wmax = 0;
    {
        std::vector<int64_t> delta(N + 1, 0);
        for (size_t t = 0; t < T; ++t)
            for (const Stay &s : stays[t]) { delta[s.first] += (int64_t)alignup(ten[t].size); delta[s.last + 1] -= (int64_t)alignup(ten[t].size); }
        int64_t live = 0;
        for (size_t i = O0; i < N; ++i) { live += delta[i]; wmax = std::max<uint64_t>(wmax, (uint64_t)live); }
    }
    const uint64_t ring_min = 2 * wmax;
    if (ring_min > ctx->budget) return fail(TGP_E_BUDGET_TOO_SMALL, "budget below twice the largest working set of one op");
    const uint64_t pin_cap = ctx->budget - ring_min;
    // pins: greedy by density score/size, exact cross products, tie -> lower id, skip what does not fit
    std::vector<int64_t> pin_off(T, -1);
    uint64_t used = 0;
    std::vector<uint32_t> cand_order;                    // pin candidates by falling density (kept for the tenants below)
    if (ctx->bits & TGP_BIT_A) {
        std::vector<uint32_t> &cand = cand_order;
        for (size_t t = 0; t < T; ++t) if (pl.score[t] > 0 && !pl.zc[t]) cand.push_back((uint32_t)t);
        std::sort(cand.begin(), cand.end(), [&](uint32_t a, uint32_t b) {
            u128 l = (u128)pl.score[a] * ten[b].size, r = (u128)pl.score[b] * ten[a].size;
            return l != r ? l > r : a < b;
        });
        for (size_t g0 = 0; g0 < cand.size();) {
            // group of equal density
            size_t g1 = g0 + 1;
            while (g1 < cand.size() && (u128)pl.score[cand[g1]] * ten[cand[g0]].size == (u128)pl.score[cand[g0]] * ten[cand[g1]].size) ++g1;
            const uint64_t cap_left = pin_cap - used;
            uint64_t total = 0;
            for (size_t k = g0; k < g1; ++k) total += alignup(ten[cand[k]].size);
            if (total > cap_left) {
                // the group does not fit: spread its pinned bytes evenly along the id order (error diffusion),
                // so the link demand of the streamed rest stays uniform over a step
                u128 err = 0;
                for (size_t k = g0; k < g1; ++k) {
                    const uint64_t a = alignup(ten[cand[k]].size);
                    err += (u128)a * cap_left;
                    if (err >= (u128)a * total) { err -= (u128)a * total; pin_off[cand[k]] = (int64_t)used; used += a; }
                }
            }
            for (size_t k = g0; k < g1; ++k) {               // whole group if it fits / greedy fill with skip
                const uint64_t a = alignup(ten[cand[k]].size);
                if (pin_off[cand[k]] < 0 && used + a <= pin_cap) { pin_off[cand[k]] = (int64_t)used; used += a; }
            }
            g0 = g1;
        }
    }
    // Pins that are resident already (a plan made in the middle of a run that keeps them): a chosen tensor that is on the
    // device keeps its place and is not loaded again; the others go, in the order they were chosen, into the first gap
    // between the kept ones that holds them (none: not pinned after all).  The pin region ends where the longer of the two
    // layouts ends.  Resident = a pin of the plan in use that was placed before the boundary, or that the plan itself kept.
    std::vector<uint8_t> kept(T, 0);
    const bool keep = first_step > 0 && ctx->replan_keep && ctx->plan.valid;
    if (keep) {
        std::vector<int64_t> res(T, -1), old_off(T, -1);
        for (auto &pin : ctx->plan.pins) old_off[pin.first] = (int64_t)pin.second;
        std::vector<int32_t> placed_at(T, -2);               // first use of the pin's own placement in the plan in use; -2: it has none
        for (const TgpCmd &c : ctx->plan.cmds)
            if (c.kind != CMD_D2H && old_off[c.tensor] >= 0 && (int64_t)c.arena_off == old_off[c.tensor] && placed_at[c.tensor] == -2) placed_at[c.tensor] = c.first_use;
        for (auto &pin : ctx->plan.pins)
            if (placed_at[pin.first] == -2 || placed_at[pin.first] < (int32_t)O0) res[pin.first] = (int64_t)pin.second;   // kept by that plan itself, or placed before the boundary
        std::vector<uint32_t> chosen;
        for (size_t t = 0; t < T; ++t) if (pin_off[t] >= 0) chosen.push_back((uint32_t)t);
        std::sort(chosen.begin(), chosen.end(), [&](uint32_t a, uint32_t b) { return pin_off[a] < pin_off[b]; });
        uint64_t region_end = used;
        std::vector<std::pair<uint64_t, uint64_t>> iv;
        for (uint32_t t : chosen)
            if (res[t] >= 0) { kept[t] = 1; iv.push_back({(uint64_t)res[t], (uint64_t)res[t] + alignup(ten[t].size)}); region_end = std::max(region_end, iv.back().second); }
        std::sort(iv.begin(), iv.end());
        std::vector<std::pair<uint64_t, uint64_t>> holes;
        uint64_t pos = 0;
        for (auto &v : iv) { if (v.first > pos) holes.push_back({pos, v.first}); pos = std::max(pos, v.second); }
        if (pos < region_end) holes.push_back({pos, region_end});
        for (uint32_t t : chosen) {
            if (kept[t]) { pin_off[t] = res[t]; continue; }
            const uint64_t a = alignup(ten[t].size);
            pin_off[t] = -1;
            for (auto &h : holes)
                if (h.second - h.first >= a) { pin_off[t] = (int64_t)h.first; h.first += a; break; }
        }
        used = region_end;
        if (ctx->budget - used < ring_min) return fail(TGP_E_BUDGET_TOO_SMALL, "kept pins leave less than the ring minimum");
    }
    for (size_t t = 0; t < T; ++t) if (pin_off[t] >= 0) { pl.pins.push_back({(uint32_t)t, (uint64_t)pin_off[t]}); if (kept[t]) pl.kept.push_back((uint32_t)t); }
    pl.ring_base = used; pl.ring_size = ctx->budget - used;
    // windowed reservation: the slot of a pinned tensor that is born on the device in a later step houses tenants until then
    std::vector<int64_t> tenant_off(T, -1);
    std::vector<int32_t> tenant_last(T, -1), landlord_wait(T, -1);
    if ((ctx->bits & TGP_BIT_W) && !pl.pins.empty() && !keep) {
        std::vector<uint8_t> written0(T, 0);
        for (size_t i = 0; i < O0; ++i)
            for (uint32_t k = 0; k < ctx->ops[i].nacc; ++k)
                if (ctx->acc[ctx->ops[i].acc0 + k].mode & TGP_W) written0[ctx->acc[ctx->ops[i].acc0 + k].tensor] = 1;
        std::vector<int32_t> first_op_of(T, -1);
        std::vector<uint32_t> first_mode(T, 0);
        for (size_t i = O0; i < N; ++i)
            for (uint32_t k = 0; k < ctx->ops[i].nacc; ++k) {
                const tgp_access &a = ctx->acc[ctx->ops[i].acc0 + k];
                if (first_op_of[a.tensor] < 0) { first_op_of[a.tensor] = (int32_t)i; first_mode[a.tensor] = a.mode; }
            }
        struct Region { uint64_t start, end, fill; uint32_t birth; int32_t wait; std::vector<uint32_t> lords; };
        std::vector<Region> regions;
        std::vector<uint32_t> late;
        for (auto &p : pl.pins) {
            const uint32_t t = p.first;
            if (ten[t].flags == TGP_T_MUTABLE && !written0[t] && first_mode[t] == TGP_W && ctx->ops[first_op_of[t]].step - first_step >= 2) late.push_back(t);
        }
        std::sort(late.begin(), late.end(), [&](uint32_t a, uint32_t b) { return pin_off[a] < pin_off[b]; });
        for (uint32_t t : late) {
            const uint64_t o = (uint64_t)pin_off[t], a = alignup(ten[t].size);
            const uint32_t b = ctx->ops[first_op_of[t]].step;
            if (!regions.empty() && regions.back().end == o && regions.back().birth == b) { regions.back().end = o + a; regions.back().lords.push_back(t); }
            else regions.push_back({o, o + a, o, b, -1, {t}});
        }
        std::stable_sort(regions.begin(), regions.end(), [](const Region &x, const Region &y) { return x.birth != y.birth ? x.birth > y.birth : x.start < y.start; });
        if (!regions.empty()) {
            // accesses of each unpinned read-only candidate, in op order (only those are ever tenants)
            std::vector<std::vector<int32_t>> acc_ops(T);
            for (size_t i = O0; i < N; ++i)
                for (uint32_t k = 0; k < ctx->ops[i].nacc; ++k) {
                    const uint32_t t = ctx->acc[ctx->ops[i].acc0 + k].tensor;
                    if (pin_off[t] < 0 && !pl.zc[t] && pl.score[t] > 0 && ten[t].flags == TGP_T_READONLY) acc_ops[t].push_back((int32_t)i);
                }
            for (uint32_t t : cand_order) {
                if (pin_off[t] >= 0 || ten[t].flags != TGP_T_READONLY) continue;
                const uint64_t a = alignup(ten[t].size);
                for (Region &r : regions) {
                    if (r.fill + a > r.end) continue;
                    int32_t first = -1, last = -1;
                    for (int32_t i : acc_ops[t]) { if (ctx->ops[i].step >= r.birth) break; if (first < 0) first = i; last = i; }
                    if (first < 0 || ctx->ops[first].step == ctx->ops[last].step) continue;      // used in fewer than two steps of the vacancy
                    tenant_off[t] = (int64_t)r.fill; tenant_last[t] = last;
                    r.fill += a;
                    r.wait = std::max(r.wait, last);
                    break;
                }
            }
            for (const Region &r : regions) for (uint32_t t : r.lords) landlord_wait[t] = r.wait;
        }
    }
    // schedule
    pl.totals.assign(ctx->steps.size() * 4, 0);
    pl.acc_where.assign(ctx->acc.size(), 0);
    pl.op_last_place.assign(N, -1);
    pl.op_is_wait_target.assign(N, 0);
    struct Slot { uint64_t start, end; int32_t last_use; };
    std::deque<Slot> fifo;
    uint64_t head = 0;
    int32_t run_wait = -1;
    std::vector<uint32_t> stay_idx(T, 0);
    std::vector<int64_t> open_at(T, -1);                 // arena offset of the open stay, -1 if none
    std::vector<uint8_t> pin_loaded(kept), written_ever(T, 0), dirty(T, 0);
    for (size_t i = 0; i < O0; ++i)                      // a tail plan: what earlier steps wrote holds data in the pool
        for (uint32_t k = 0; k < ctx->ops[i].nacc; ++k)
            if (ctx->acc[ctx->ops[i].acc0 + k].mode & TGP_W) written_ever[ctx->acc[ctx->ops[i].acc0 + k].tensor] = 1;
    std::vector<int32_t> last_wb(T, -1);
    std::vector<std::vector<uint32_t>> ending(N);
    auto emit = [&](uint8_t kind, uint32_t t, uint64_t where, int32_t wait, int32_t first, int32_t rel) {
        pl.cmds.push_back({(uint32_t)pl.cmds.size(), kind, t, ten[t].size, ten[t].off, where, wait, first, rel});
        uint64_t *tot = &pl.totals[ctx->ops[first].step * 4];
        tot[3] += 1;
        if (kind == CMD_H2D) tot[0] += ten[t].size; else if (kind == CMD_D2H) tot[1] += ten[t].size;
        if (kind != CMD_D2H) pl.op_last_place[first] = (int32_t)pl.cmds.size() - 1;
    };
    for (size_t i = O0; i < N; ++i) {
        const TgpOp &o = ctx->ops[i];
        for (uint32_t k = 0; k < o.nacc; ++k) {
            const tgp_access &a = ctx->acc[o.acc0 + k];
            uint32_t t = a.tensor;
            if (pl.zc[t]) { pl.totals[o.step * 4 + 2] += a.touched_bytes; pl.acc_where[o.acc0 + k] = UINT64_MAX; continue; }
            bool mut = ten[t].flags == TGP_T_MUTABLE;
            bool fresh = mut && a.mode == TGP_W && !written_ever[t];
            if (pin_off[t] >= 0) {
                if (!pin_loaded[t]) {
                    pin_loaded[t] = 1;
                    emit(fresh ? CMD_ALLOC : CMD_H2D, t, (uint64_t)pin_off[t], landlord_wait[t], (int32_t)i, (int32_t)N - 1);
                    if (landlord_wait[t] >= 0) pl.op_is_wait_target[landlord_wait[t]] = 1;
                }
                pl.acc_where[o.acc0 + k] = (uint64_t)pin_off[t];
            } else if (tenant_off[t] >= 0 && (int32_t)i <= tenant_last[t]) {
                // a tenant of a late-born pinned tensor's slot: loaded once, used there until its last access of the vacancy
                if (!pin_loaded[t]) { pin_loaded[t] = 1; emit(CMD_H2D, t, (uint64_t)tenant_off[t], -1, (int32_t)i, tenant_last[t]); }
                pl.acc_where[o.acc0 + k] = (uint64_t)tenant_off[t];
            } else {
                if (open_at[t] < 0) {
                    while (stays[t][stay_idx[t]].first < (int32_t)i) stay_idx[t]++;      // stays a tenancy made unnecessary
                    const Stay &s = stays[t][stay_idx[t]];
                    uint64_t sz = alignup(ten[t].size);
                    if (sz > pl.ring_size) return fail(TGP_E_BUDGET_TOO_SMALL, "tensor larger than the ring");
                    int32_t ev = -1;
                    if (head + sz > pl.ring_size) {                      // tail too short: skip it and wrap
                        while (!fifo.empty() && fifo.front().start >= head) { ev = std::max(ev, fifo.front().last_use); fifo.pop_front(); }
                        head = 0;
                    }
                    while (!fifo.empty() && fifo.front().start < head + sz && fifo.front().end > head) { ev = std::max(ev, fifo.front().last_use); fifo.pop_front(); }
                    run_wait = std::max(run_wait, std::max(ev, last_wb[t]));
                    if (run_wait >= (int32_t)i) return fail(TGP_E_BUDGET_TOO_SMALL, "ring too small: a stay would wait on its own op");
                    fifo.push_back({head, head + sz, s.last});
                    open_at[t] = (int64_t)(pl.ring_base + head);
                    emit(fresh ? CMD_ALLOC : CMD_H2D, t, pl.ring_base + head, run_wait, (int32_t)i, s.last);
                    if (run_wait >= 0) pl.op_is_wait_target[run_wait] = 1;
                    ending[s.last].push_back(t);
                    head += sz;
                }
                pl.acc_where[o.acc0 + k] = (uint64_t)open_at[t];
            }
            if (a.mode & TGP_W) { written_ever[t] = 1; if (pin_off[t] < 0) dirty[t] = 1; }
        }
        for (uint32_t t : ending[i]) {
            uint64_t where = (uint64_t)open_at[t];
            open_at[t] = -1;
            if (dirty[t]) { dirty[t] = 0; emit(CMD_D2H, t, where, (int32_t)i, (int32_t)i, (int32_t)i); last_wb[t] = (int32_t)i; pl.op_is_wait_target[i] = 1; }
            stay_idx[t]++;
        }
    }
    pl.valid = true;
    out = std::move(pl);
    return TGP_OK;
}

extern "C" {

int tgp_plan(tgp_ctx *ctx) {
    if (!ctx) return TGP_E_INVAL;
    if (!ctx->traced) return tgp_fail(ctx, TGP_E_STATE, "no finished trace");
    if (!ctx->budget) return tgp_fail(ctx, TGP_E_STATE, "no budget set");
    if (ctx->steps.empty() || ctx->ops.empty()) return tgp_fail(ctx, TGP_E_STATE, "empty trace");
    if (ctx->replan_thread.joinable()) ctx->replan_thread.join();
    ctx->tail_ready = false;
    ctx->base_plan = TgpPlan();
    TgpPlan pl;
    std::string err;
    const int rc = build_plan(ctx, 0, pl, err);
    if (rc) return tgp_fail(ctx, rc, err);
    ctx->plan = std::move(pl);
    return TGP_OK;
}

int tgp_replan_begin(tgp_ctx *ctx, uint32_t first_step, const uint64_t *op_ns, uint64_t n_ops) {
    if (!ctx) return TGP_E_INVAL;
    if (!ctx->plan.valid) return TGP_E_NO_PLAN;
    if (ctx->variant != TGP_VAR_EXPLICIT_RING) return tgp_fail(ctx, TGP_E_STATE, "only the explicit engine re-plans in the middle of a run");
    if (!first_step || first_step >= ctx->steps.size()) return tgp_fail(ctx, TGP_E_INVAL, "the boundary must lie between two steps of the trace");
    if (first_step <= ctx->plan.first_step) return tgp_fail(ctx, TGP_E_INVAL, "the boundary must lie after the current plan's first step");
    if (n_ops && (!op_ns || n_ops != ctx->ops.size())) return tgp_fail(ctx, TGP_E_INVAL, "one time per op of the whole trace is required");
    if (ctx->replan_thread.joinable()) return tgp_fail(ctx, TGP_E_STATE, "a re-plan is already under way");
    // the log is stored without touching the plan in use (tgp_set_measured_times() would invalidate it)
    if (n_ops) ctx->measured_ns.assign(op_ns, op_ns + n_ops);
    ctx->tail_ready = false; ctx->tail_rc = TGP_OK; ctx->tail_err.clear(); ctx->tail_step = first_step;
    ctx->replan_thread = std::thread([ctx, first_step]() { ctx->tail_rc = build_plan(ctx, first_step, ctx->tail_plan, ctx->tail_err); });
    return TGP_OK;
}

int tgp_replan_wait(tgp_ctx *ctx) {
    if (!ctx) return TGP_E_INVAL;
    if (!ctx->replan_thread.joinable()) return ctx->tail_ready ? TGP_OK : tgp_fail(ctx, TGP_E_STATE, "no re-plan under way");
    ctx->replan_thread.join();
    if (ctx->tail_rc) return tgp_fail(ctx, ctx->tail_rc, "re-plan: " + ctx->tail_err);
    ctx->tail_ready = true;
    return TGP_OK;
}

int tgp_plan_export(const tgp_ctx *ctx, uint32_t what, void *buf, uint64_t *bytes) {
    if (!ctx) return TGP_E_INVAL;
    const bool tail = what & TGP_X_TAIL;
    what &= ~TGP_X_TAIL;
    if (tail && (!ctx->tail_ready || !ctx->tail_plan.valid)) return TGP_E_NO_PLAN;
    if (!tail && !ctx->plan.valid) return TGP_E_NO_PLAN;
    const TgpPlan &pl = tail ? ctx->tail_plan : ctx->plan;
    std::vector<uint8_t> b;
    switch (what) {
    case TGP_X_CLASSES: b.assign(pl.cls.begin() + pl.first_op, pl.cls.end()); break;
    case TGP_X_TENSORS:
        for (size_t t = 0; t < pl.crit.size(); ++t) { put<uint8_t>(b, pl.crit[t]); put<uint8_t>(b, pl.zc[t]); put<uint64_t>(b, pl.score[t]); }
        break;
    case TGP_X_PINS:
        for (auto &p : pl.pins) { put<uint32_t>(b, p.first); put<uint64_t>(b, p.second); }
        put<uint64_t>(b, pl.ring_base); put<uint64_t>(b, pl.ring_size);
        break;
    case TGP_X_COMMANDS:
        b.reserve(pl.cmds.size() * 45);
        for (const TgpCmd &c : pl.cmds) {
            put<uint32_t>(b, c.seq); put<uint8_t>(b, c.kind); put<uint32_t>(b, c.tensor); put<uint64_t>(b, c.bytes);
            put<uint64_t>(b, c.pool_off); put<uint64_t>(b, c.arena_off); put<int32_t>(b, c.wait_op);
            put<int32_t>(b, c.first_use); put<int32_t>(b, c.release_after);
        }
        break;
    case TGP_X_TOTALS:
        for (size_t k = (size_t)pl.first_step * 4; k < pl.totals.size(); ++k) put<uint64_t>(b, pl.totals[k]);
        break;
    default: return TGP_E_INVAL;
    }
    return give(b, buf, bytes);
}

}  // extern "C"
