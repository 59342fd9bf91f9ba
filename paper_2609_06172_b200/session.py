"""Convenience layer over the binding: registers a sub-allocated pool, binds the decoder and plans.

Marshalling only.  `layout` is any object with the attributes the synthetic-input module produces
(.cfg, .tensors[...] with kind/layer/expert/block/row0/rows/pool_off/size/flags/site_hash, .pool_bytes,
.budget); nothing here computes a forward pass or a schedule.
"""
from __future__ import annotations

import numpy as np

from . import binding as tb


def model_cfg(cfg) -> tb.ModelCfg:
    return tb.ModelCfg(cfg.L, cfg.d, cfg.Hq, cfg.Hkv, cfg.Dh, cfg.F, cfg.V, cfg.E, cfg.topk, cfg.B, cfg.max_len, cfg.TK,
                       cfg.rope_base, cfg.eps)


class Session:
    """Registry + model binding for one pool.  pool_base: address of the host pool (int), or None for planning
    only (a dummy 512-aligned address is registered: planning never dereferences it)."""

    def __init__(self, layout, machine: dict, pool_base=None, pool_flags=tb.POOL_PLAIN, router_bias=None):
        self.layout = layout
        self.ctx = tb.Ctx(**machine)
        base = pool_base if pool_base is not None else 1 << 30
        self.pool = self.ctx.pool_register(base, layout.pool_bytes, pool_flags)
        self.roles = []
        for t in layout.tensors:
            tid = self.ctx.tensor_register(self.pool, t.pool_off, t.size, t.site_hash, t.layer, t.kind, t.flags)
            assert tid == t.tid
            is_tile = t.kind in (tb.K_KTILE, tb.K_VTILE)                 # a KV tile is [B * Hkv * TK rows, Dh]
            rows = layout.cfg.B * layout.cfg.Hkv * layout.cfg.TK if is_tile else t.rows
            self.roles.append((t.kind, t.layer, t.expert, t.block, t.row0, rows, tid))
        self.cfg = model_cfg(layout.cfg)
        self.router_bias = router_bias
        self.ctx.model_bind(self.cfg, self.roles, router_bias)
        self.ctx.set_budget(layout.budget)

    def plan(self, S=None, T=None, expert_counts=None, variant=tb.VAR_EXPLICIT_RING, bits=tb.BIT_A | tb.BIT_P | tb.BIT_ZC | tb.BIT_W):
        cfg = self.layout.cfg
        self.ctx.set_variant(variant, bits)
        self.ctx.model_trace(cfg.S if S is None else S, cfg.T if T is None else T, expert_counts)
        self.ctx.plan()
        return self.ctx.plan_blobs()

    def attach_device(self, arena, arena_bytes, workspace, ws_bytes, max_tokens):
        self.ctx.set_arena(arena, arena_bytes)
        self.ctx.model_bind(self.cfg, self.roles, self.router_bias, workspace, ws_bytes, max_tokens)

    def close(self):
        self.ctx.close()
