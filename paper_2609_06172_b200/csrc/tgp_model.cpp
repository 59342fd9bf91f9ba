// Model binding (which registered sub-range plays which role) and the library's own analytic op
// trace for the bound decoder.  Host only.
//
// Cost table per op, integers (M = tokens in the step, pos0 = cached tokens before it, kvlen = pos0 + q):
//   embed      0 flops,                     6*M*d bytes,                       table R, touched 2*M*d
//   rmsnorm    4*m*d,                        6*m*d + 2*d,                       gain R
//   gemm block 2*m*K*n,                      2*m*K + 2*K*n + 4*m*n (+4*m*n residual),  block R, touched = its size
//   rope+kv    6*M*(Hq+Hkv)*Dh,              6*M*(Hq+2*Hkv)*Dh,                 tiles of the new tokens W (K then V)
//   attention  4*B*Hq*Dh*(tri(kvlen)-tri(pos0)),  4*M*Hq*Dh + 4*B*Hkv*kvlen*Dh, tiles holding valid tokens R (K then V)
//   swiglu     8*m*F,                        10*m*F
//   router     2*M*d*E,                      2*M*d + 2*d*E + 4*M*E,             router R
//   argmax     B*V,                          4*B*V + 4*B
#include "tgp_internal.h"
#include <algorithm>

static inline uint64_t site_of(uint32_t op_kind, uint32_t sub) { return ((uint64_t)op_kind << 8) | sub; }
static inline uint64_t tri(uint64_t n) { return n * (n + 1) / 2; }

struct RoleIndex {
    std::map<std::tuple<uint32_t, int32_t, int32_t>, std::vector<uint32_t>> m;   // (kind, layer, expert) -> role ids by block
    const std::vector<uint32_t> *get(uint32_t kind, int32_t layer, int32_t expert) const {
        auto it = m.find(std::make_tuple(kind, layer, expert));
        return it == m.end() ? nullptr : &it->second;
    }
};

static RoleIndex build_index(const tgp_ctx *ctx) {
    RoleIndex ix;
    for (uint32_t r = 0; r < ctx->roles.size(); ++r) ix.m[std::make_tuple(ctx->roles[r].kind, ctx->roles[r].layer, ctx->roles[r].expert)].push_back(r);
    for (auto &kv : ix.m)
        std::sort(kv.second.begin(), kv.second.end(), [&](uint32_t a, uint32_t b) { return ctx->roles[a].block < ctx->roles[b].block; });
    return ix;
}

extern "C" int tgp_model_trace(tgp_ctx *ctx, uint32_t S, uint32_t T, const uint32_t *expert_counts) {
    if (!ctx) return TGP_E_INVAL;
    if (!ctx->bound) return tgp_fail(ctx, TGP_E_STATE, "no model bound");
    const tgp_model_cfg &c = ctx->cfg;
    if (S == 0 || S + T > c.max_len) return tgp_fail(ctx, TGP_E_INVAL, "S + T exceeds max_len");
    if (c.E && !expert_counts) return tgp_fail(ctx, TGP_E_INVAL, "an MoE trace needs the routed-token counts");
    RoleIndex ix = build_index(ctx);
    int rc = tgp_trace_begin(ctx);
    if (rc) return rc;
    const uint64_t B = c.B, d = c.d, Hq = c.Hq, Hkv = c.Hkv, Dh = c.Dh, F = c.F, V = c.V, TK = c.TK, E = c.E;
    std::vector<tgp_access> acc;
    auto need = [&](uint32_t kind, int32_t layer, int32_t expert) -> const std::vector<uint32_t> * {
        const std::vector<uint32_t> *v = ix.get(kind, layer, expert);
        if (!v) tgp_fail(ctx, TGP_E_STATE, "a tensor role of the model is not bound");
        return v;
    };
#define NEED(var, kind, layer, expert) const std::vector<uint32_t> *var = need(kind, layer, expert); if (!var) return TGP_E_STATE;
#define EMIT(site, layer, kind, flops, hbm) do { rc = tgp_trace_op(ctx, site, layer, kind, flops, hbm, (uint32_t)acc.size(), acc.data()); if (rc) return rc; } while (0)
    for (uint32_t k = 0; k <= T; ++k) {
        const uint64_t q = k == 0 ? S : 1, pos0 = k == 0 ? 0 : S + k - 1, M = B * q, kvlen = pos0 + q;
        rc = tgp_trace_step(ctx, k == 0 ? TGP_PREFILL : TGP_DECODE);
        if (rc) return rc;
        auto gemm_blocks = [&](uint32_t kind, int32_t layer, int32_t expert, uint64_t m, bool residual) -> int {
            NEED(blk, kind, layer, expert);
            for (uint32_t r : *blk) {
                const TgpTensor &t = ctx->tensors[ctx->roles[r].tensor];
                uint64_t n = ctx->roles[r].rows, K = t.size / (2 * n);
                acc.assign(1, tgp_access{ctx->roles[r].tensor, TGP_R, t.size});
                EMIT(site_of(TGP_OP_GEMM, kind), layer, TGP_OP_GEMM, 2 * m * K * n, 2 * m * K + 2 * K * n + 4 * m * n + (residual ? 4 * m * n : 0));
            }
            return TGP_OK;
        };
        auto norm = [&](uint32_t kind, int32_t layer, uint64_t m) -> int {
            NEED(g, kind, layer, -1);
            acc.assign(1, tgp_access{ctx->roles[(*g)[0]].tensor, TGP_R, 2 * d});
            EMIT(site_of(TGP_OP_RMSNORM, kind), layer, TGP_OP_RMSNORM, 4 * m * d, m * d * 6 + 2 * d);
            return TGP_OK;
        };
        {
            NEED(emb, TGP_K_EMBED, -1, -1);
            acc.assign(1, tgp_access{ctx->roles[(*emb)[0]].tensor, TGP_R, M * d * 2});
            EMIT(site_of(TGP_OP_EMBED, 0), -1, TGP_OP_EMBED, 0, M * d * 6);
        }
        for (int32_t l = 0; l < (int32_t)c.L; ++l) {
            if ((rc = norm(TGP_K_G1, l, M))) return rc;
            if ((rc = gemm_blocks(TGP_K_WQ, l, -1, M, false))) return rc;
            if ((rc = gemm_blocks(TGP_K_WK, l, -1, M, false))) return rc;
            if ((rc = gemm_blocks(TGP_K_WV, l, -1, M, false))) return rc;
            NEED(kt, TGP_K_KTILE, l, -1);
            NEED(vt, TGP_K_VTILE, l, -1);
            const uint64_t j_last = (kvlen - 1) / TK;
            if (kt->size() <= j_last || vt->size() <= j_last) return tgp_fail(ctx, TGP_E_STATE, "not enough KV tiles bound");
            acc.clear();
            for (const std::vector<uint32_t> *tiles : {kt, vt})
                for (uint64_t j = pos0 / TK; j <= j_last; ++j) {
                    uint64_t ntok = std::min(kvlen, (j + 1) * TK) - std::max(pos0, j * TK);
                    acc.push_back({ctx->roles[(*tiles)[j]].tensor, TGP_W, B * Hkv * ntok * Dh * 2});
                }
            EMIT(site_of(TGP_OP_ROPE_KV, 0), l, TGP_OP_ROPE_KV, 6 * M * (Hq + Hkv) * Dh, M * (Hq + 2 * Hkv) * Dh * 6);
            acc.clear();
            for (const std::vector<uint32_t> *tiles : {kt, vt})
                for (uint64_t j = 0; j <= j_last; ++j) {
                    uint64_t valid = std::min(kvlen, (j + 1) * TK) - j * TK;
                    acc.push_back({ctx->roles[(*tiles)[j]].tensor, TGP_R, B * Hkv * valid * Dh * 2});
                }
            EMIT(site_of(TGP_OP_ATTN, 0), l, TGP_OP_ATTN, 4 * B * Hq * Dh * (tri(kvlen) - tri(pos0)), 4 * M * Hq * Dh + 4 * B * Hkv * kvlen * Dh);
            if ((rc = gemm_blocks(TGP_K_WO, l, -1, M, true))) return rc;
            if ((rc = norm(TGP_K_G2, l, M))) return rc;
            if (E == 0) {
                if ((rc = gemm_blocks(TGP_K_WG, l, -1, M, false))) return rc;
                if ((rc = gemm_blocks(TGP_K_WU, l, -1, M, false))) return rc;
                acc.clear();
                EMIT(site_of(TGP_OP_SWIGLU, 0), l, TGP_OP_SWIGLU, 8 * M * F, M * F * 10);
                if ((rc = gemm_blocks(TGP_K_WD, l, -1, M, true))) return rc;
            } else {
                NEED(rt, TGP_K_ROUTER, l, -1);
                const TgpTensor &t = ctx->tensors[ctx->roles[(*rt)[0]].tensor];
                acc.assign(1, tgp_access{ctx->roles[(*rt)[0]].tensor, TGP_R, t.size});
                EMIT(site_of(TGP_OP_ROUTER, 0), l, TGP_OP_ROUTER, 2 * M * d * E, 2 * M * d + 2 * d * E + 4 * M * E);
                for (int32_t e = 0; e < (int32_t)E; ++e) {
                    uint64_t me = expert_counts[((uint64_t)k * c.L + l) * E + e];
                    if (!me) continue;
                    if ((rc = gemm_blocks(TGP_K_WG, l, e, me, false))) return rc;
                    if ((rc = gemm_blocks(TGP_K_WU, l, e, me, false))) return rc;
                    acc.clear();
                    EMIT(site_of(TGP_OP_SWIGLU, 0), l, TGP_OP_SWIGLU, 8 * me * F, me * F * 10);
                    if ((rc = gemm_blocks(TGP_K_WD, l, e, me, true))) return rc;
                }
            }
        }
        if ((rc = norm(TGP_K_GF, -1, B))) return rc;
        if ((rc = gemm_blocks(TGP_K_LM, -1, -1, B, false))) return rc;
        acc.clear();
        EMIT(site_of(TGP_OP_ARGMAX, 0), -1, TGP_OP_ARGMAX, B * V, 4 * B * V + 4 * B);
    }
#undef NEED
#undef EMIT
    return tgp_trace_end(ctx);
}
