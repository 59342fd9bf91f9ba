"""Oracle forward pass: decoder-only transformer, prefill and decode, in numpy.

TEST INFRASTRUCTURE - see oracle/__init__.py.

What is computed (the workload the paper runs under oversubscription, Section V-A:
LLM inference; operator families named in Section III-C: GEMM/GEMV, elementwise /
normalisation, attention).  Precision contract of this build (the paper states none):
bf16 (round-to-nearest-even) at weights, the KV cache and every GEMM input activation;
everything else (residual stream, accumulators, norm statistics, softmax, router,
logits) is fp32 on the GPU.  The oracle accumulates in ``dtype`` (float64 by default)
and rounds once to fp32 at the points where the GPU holds an fp32 value.

No blocking, fusion or reordering: each step below is the textbook definition.
"""
from __future__ import annotations

import numpy as np


def to_f32(x):
    return np.asarray(x).astype(np.float32)


def bf16_round(x):
    """Round to fp32, then round-to-nearest-even to bf16; returns fp32 values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bits_to_float(bits, dtype):
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(dtype)


def rope_table(Dh, max_pos, base):
    """cos/sin tables [max_pos, Dh/2]: angle = pos * base**(-2i/Dh) in double, cast to fp32."""
    i = np.arange(Dh // 2, dtype=np.float64)
    inv = base ** (-2.0 * i / Dh)
    ang = np.arange(max_pos, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


class OracleModel:
    """weights: dict (kind, layer, expert) -> uint16 bf16 bits [out, in]; kinds by integer as in the layout."""

    # kind ids (kept literal so this file depends on nothing else)
    EMBED, G1, WQ, WK, WV, WO, G2, WG, WU, WD, GF, LM, ROUTER = range(13)

    def __init__(self, cfg, weights_bits, router_bias=None, dtype=np.float64):
        self.cfg = cfg
        self.dt = dtype
        self.w = {k: bits_to_float(v, dtype) for k, v in weights_bits.items()}
        self.bias = None if router_bias is None else np.asarray(router_bias, dtype=np.float32)
        self.cos, self.sin = rope_table(cfg.Dh, cfg.max_len, cfg.rope_base)
        self.K = np.zeros((cfg.L, cfg.B, cfg.Hkv, cfg.max_len, cfg.Dh), dtype=dtype)
        self.V = np.zeros_like(self.K)
        self.expert_counts = []          # per step: [L][E] token counts (MoE only)
        # optional hook(name, layer, pre, rounded) -> array to continue with, called at every bf16 rounding point with
        # the fp32 value before rounding and the oracle's rounding of it (used by the lockstep parity test)
        self.hook = None

    # ---- pieces -------------------------------------------------------------------------
    def _round(self, name, layer, pre):
        pre = to_f32(pre)
        out = bf16_round(pre)
        if self.hook is not None:
            out = np.asarray(self.hook(name, layer, pre, out), dtype=np.float32)
        return out

    def rmsnorm(self, x, g, name="h", layer=-1):
        """bf16( x / sqrt(mean(x^2) + eps) * g ) per row."""
        xd = x.astype(self.dt)
        ms = np.mean(xd * xd, axis=-1, keepdims=True)
        return self._round(name, layer, xd / np.sqrt(ms + self.cfg.eps) * g).astype(self.dt)

    def linear(self, a, W):
        """fp32( a @ W^T ), W stored [out, in]."""
        return to_f32(a.astype(self.dt) @ W.T)

    def rope(self, t, pos0):
        """t: [B, q, H, Dh] fp32 values; rotate pairs (i, i + Dh/2) by the position's angle."""
        q = t.shape[1]
        half = self.cfg.Dh // 2
        c = self.cos[pos0:pos0 + q][None, :, None, :].astype(self.dt)
        s = self.sin[pos0:pos0 + q][None, :, None, :].astype(self.dt)
        a, b = t[..., :half].astype(self.dt), t[..., half:].astype(self.dt)
        return to_f32(np.concatenate([a * c - b * s, b * c + a * s], axis=-1))

    def attention(self, l, qb, pos0):
        """qb: [B, q, Hq, Dh] bf16-valued.  Causal softmax(q K^T / sqrt(Dh)) V over the cache."""
        cfg = self.cfg
        B, q = qb.shape[0], qb.shape[1]
        kvlen = pos0 + q
        grp = cfg.Hq // cfg.Hkv
        scale = np.float32(1.0 / np.sqrt(np.float64(cfg.Dh)))
        out = np.empty((B, q, cfg.Hq, cfg.Dh), dtype=np.float32)
        keypos = np.arange(kvlen)[None, :]
        qpos = (pos0 + np.arange(q))[:, None]
        mask = keypos <= qpos
        for b in range(B):
            for h in range(cfg.Hq):
                Kh = self.K[l, b, h // grp, :kvlen]
                Vh = self.V[l, b, h // grp, :kvlen]
                s = to_f32(qb[b, :, h].astype(self.dt) @ Kh.T).astype(self.dt) * self.dt(scale)
                s = np.where(mask, s, -np.inf)
                p = np.exp(s - s.max(axis=-1, keepdims=True))
                p = p / p.sum(axis=-1, keepdims=True)
                out[b, :, h] = to_f32(p @ Vh)
        return out

    def ffn_dense(self, l, h2, e=-1):
        g = self.linear(h2, self.w[(self.WG, l, e)]).astype(self.dt)
        u = self.linear(h2, self.w[(self.WU, l, e)]).astype(self.dt)
        a = self._round("a" if e < 0 else "a.e%d" % e, l, g / (1.0 + np.exp(-g)) * u)
        return self.linear(a, self.w[(self.WD, l, e)])

    def ffn_moe(self, l, h2, x):
        """Router -> top-2 (tie: lower id) -> softmax over the two logits -> experts in ascending id."""
        cfg = self.cfg
        M = h2.shape[0]
        logits = to_f32(self.linear(h2, self.w[(self.ROUTER, l, -1)]).astype(self.dt) + self.bias[l].astype(self.dt))
        order = np.argsort(-logits, axis=-1, kind="stable")[:, :cfg.topk]       # stable: ties keep lower id first
        sel = np.take_along_axis(logits, order, axis=-1).astype(self.dt)
        ex = np.exp(sel - sel.max(axis=-1, keepdims=True))
        gates = to_f32(ex / ex.sum(axis=-1, keepdims=True))
        counts = np.zeros(cfg.E, dtype=np.int64)
        for e in range(cfg.E):
            rows, slot = np.nonzero(order == e)
            counts[e] = len(rows)
            if len(rows) == 0:
                continue
            y = self.ffn_dense(l, h2[rows], e)
            x[rows] = to_f32(x[rows].astype(self.dt) + to_f32(gates[rows, slot][:, None].astype(self.dt) * y.astype(self.dt)).astype(self.dt))
        return x, counts

    # ---- one step -----------------------------------------------------------------------
    def step(self, tokens, pos0, all_positions=False):
        """tokens [B, q] int; appends q positions to the cache at pos0; returns fp32 logits [B, V]
        (last position) or [B, q, V]."""
        cfg = self.cfg
        tokens = np.asarray(tokens)
        B, q = tokens.shape
        x = to_f32(self.w[(self.EMBED, -1, -1)][tokens])                      # [B, q, d]
        counts_step = []
        for l in range(cfg.L):
            h = self.rmsnorm(x, self.w[(self.G1, l, -1)][0], "h", l)
            qv = self.linear(h, self.w[(self.WQ, l, -1)]).reshape(B, q, cfg.Hq, cfg.Dh)
            kv = self.linear(h, self.w[(self.WK, l, -1)]).reshape(B, q, cfg.Hkv, cfg.Dh)
            vv = self.linear(h, self.w[(self.WV, l, -1)]).reshape(B, q, cfg.Hkv, cfg.Dh)
            qb = self._round("q", l, self.rope(qv, pos0))
            kb = self._round("k", l, self.rope(kv, pos0))
            vb = self._round("v", l, vv)
            self.K[l, :, :, pos0:pos0 + q] = kb.transpose(0, 2, 1, 3)
            self.V[l, :, :, pos0:pos0 + q] = vb.transpose(0, 2, 1, 3)
            o = self._round("o", l, self.attention(l, qb, pos0)).reshape(B, q, cfg.Hq * cfg.Dh)
            x = to_f32(x.astype(self.dt) + self.linear(o, self.w[(self.WO, l, -1)]).astype(self.dt))
            h2 = self.rmsnorm(x, self.w[(self.G2, l, -1)][0], "h2", l)
            if cfg.E == 0:
                x = to_f32(x.astype(self.dt) + self.ffn_dense(l, h2).astype(self.dt))
            else:
                xf, c = self.ffn_moe(l, h2.reshape(B * q, cfg.d), x.reshape(B * q, cfg.d).copy())
                x = xf.reshape(B, q, cfg.d)
                counts_step.append(c)
        self.expert_counts.append(counts_step)
        xs = x if all_positions else x[:, -1:, :]
        hf = self.rmsnorm(xs, self.w[(self.GF, -1, -1)][0], "hf", -1)
        logits = self.linear(hf, self.w[(self.LM, -1, -1)])
        return logits if all_positions else logits[:, 0, :]

    def generate(self, prompt, n_decode, forced=None):
        """Prefill + n_decode greedy steps (argmax, tie -> lowest id).  Returns (logits per step, tokens [B, n_decode])."""
        logits = [self.step(prompt, 0)]
        toks = []
        pos = prompt.shape[1]
        for t in range(n_decode):
            nxt = np.argmax(logits[-1], axis=-1).astype(np.int32) if forced is None else np.asarray(forced)[:, t]
            toks.append(nxt)
            logits.append(self.step(nxt[:, None], pos))
            pos += 1
        return logits, (np.stack(toks, axis=1) if toks else np.zeros((prompt.shape[0], 0), np.int32))
