"""Pins for the oracle forward pass: brute-force scalar loops in double, closed forms,
special cases that reduce to textbook routines, and library cross-checks - chosen so that a
dropped term, a wrong sign or index, or a transposed operand fails at least one of them."""
import math
import struct
from dataclasses import replace

import numpy as np
import pytest

import seeded_inputs as si
from oracle.forward import OracleModel, bf16_round, rope_table

TOY = si.ModelConfig("toy", L=2, d=16, Hq=4, Hkv=2, Dh=4, F=24, V=40, B=2, S=5, T=3, TK=4, seed=99, budget_rule="half_w")


def toy_model(cfg=TOY, dtype=np.float64, scale_up=8.0):
    lay = si.build_layout(cfg)
    wb = si.weights_as_bits(lay)
    # enlarge the toy weights (std 0.02 at d=16 gives vanishing signals); stays exactly bf16
    for k, v in wb.items():
        if k[0] not in (si.K_G1, si.K_G2, si.K_GF):
            wb[k] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(v) * np.float32(scale_up))
    return OracleModel(cfg, wb, si.router_bias(cfg), dtype=dtype), wb


# ---------- scalar reference: python floats (double), explicit loops, struct-based bf16 rounding ------------
def s_f32(x):
    return struct.unpack("<f", struct.pack("<f", x))[0]


def s_bf16(x):
    u = struct.unpack("<I", struct.pack("<f", x))[0]
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return struct.unpack("<f", struct.pack("<I", u))[0]


def scalar_forward(cfg, W, tokens_b, bias=None, routed=None):
    """One sequence, prefill of all its tokens; returns logits for every position (lists of python floats).
    With cfg.E > 0 the FFN is the mixture of experts: router logits = h2 . Wr + bias in fp32, the two largest (tie ->
    lower id), gates = softmax over those two logits only, each chosen expert's SwiGLU FFN scaled by its gate after the
    down projection (fp32) and added to the residual stream in ascending expert id.  routed (a list) receives the
    (layer, position, [(expert, gate)]) choices."""
    f = lambda k, l=-1, e=-1: si.bf16_bits_to_f32(W[(k, l, e)]).astype(np.float64).tolist()
    S = len(tokens_b)
    half = cfg.Dh // 2
    x = [[s_f32(v) for v in f(si.K_EMBED)[t]] for t in tokens_b]

    def rms(row, g):
        ms = sum(v * v for v in row) / len(row)
        return [s_bf16(v / math.sqrt(ms + cfg.eps) * gi) for v, gi in zip(row, g)]

    def lin(row, Wm):          # Wm [out][in]
        return [s_f32(sum(row[i] * Wm[o][i] for i in range(len(row)))) for o in range(len(Wm))]

    def rope(vec, p):          # one head
        out = [0.0] * cfg.Dh
        for i in range(half):
            ang = p * cfg.rope_base ** (-2.0 * i / cfg.Dh)
            c, s = s_f32(math.cos(ang)), s_f32(math.sin(ang))
            out[i] = s_f32(vec[i] * c - vec[i + half] * s)
            out[i + half] = s_f32(vec[i + half] * c + vec[i] * s)
        return out

    for l in range(cfg.L):
        Kc, Vc, Q = [], [], []
        for p in range(S):
            h = rms(x[p], f(si.K_G1, l)[0])
            q, k, v = lin(h, f(si.K_WQ, l)), lin(h, f(si.K_WK, l)), lin(h, f(si.K_WV, l))
            Q.append([[s_bf16(z) for z in rope(q[hh * cfg.Dh:(hh + 1) * cfg.Dh], p)] for hh in range(cfg.Hq)])
            Kc.append([[s_bf16(z) for z in rope(k[hh * cfg.Dh:(hh + 1) * cfg.Dh], p)] for hh in range(cfg.Hkv)])
            Vc.append([[s_bf16(z) for z in v[hh * cfg.Dh:(hh + 1) * cfg.Dh]] for hh in range(cfg.Hkv)])
        scale = s_f32(1.0 / math.sqrt(cfg.Dh))
        for p in range(S):
            o = []
            for hh in range(cfg.Hq):
                g = hh // (cfg.Hq // cfg.Hkv)
                sc = [s_f32(sum(Q[p][hh][i] * Kc[j][g][i] for i in range(cfg.Dh))) * scale for j in range(p + 1)]
                mx = max(sc)
                e = [math.exp(z - mx) for z in sc]
                den = sum(e)
                o += [s_bf16(s_f32(sum(e[j] / den * Vc[j][g][i] for j in range(p + 1)))) for i in range(cfg.Dh)]
            att = lin(o, f(si.K_WO, l))
            x[p] = [s_f32(a + b) for a, b in zip(x[p], att)]
            h2 = rms(x[p], f(si.K_G2, l)[0])

            def ffn(e):
                gt, up = lin(h2, f(si.K_WG, l, e)), lin(h2, f(si.K_WU, l, e))
                a = [s_bf16(s_f32(gv / (1.0 + math.exp(-gv)) * uv)) for gv, uv in zip(gt, up)]
                return lin(a, f(si.K_WD, l, e))

            if not cfg.E:
                x[p] = [s_f32(a_ + b_) for a_, b_ in zip(x[p], ffn(-1))]
                continue
            rl = [s_f32(z + float(bias[l][e])) for e, z in enumerate(lin(h2, f(si.K_ROUTER, l)))]
            first = max(range(cfg.E), key=lambda e: (rl[e], -e))                       # largest logit, lower id on a tie
            second = max((e for e in range(cfg.E) if e != first), key=lambda e: (rl[e], -e))
            mx = max(rl[first], rl[second])
            w1, w2 = math.exp(rl[first] - mx), math.exp(rl[second] - mx)
            gate = {first: s_f32(w1 / (w1 + w2)), second: s_f32(w2 / (w1 + w2))}
            if routed is not None:
                routed.append((l, p, sorted(gate.items())))
            for e in sorted(gate):                                                     # ascending expert id
                y = ffn(e)
                x[p] = [s_f32(a_ + s_f32(gate[e] * b_)) for a_, b_ in zip(x[p], y)]
    return [lin(rms(x[p], f(si.K_GF)[0]), f(si.K_LM)) for p in range(S)]


def test_matches_scalar_loops():
    m, W = toy_model()
    toks = si.prompt_tokens(TOY)
    got = m.step(toks, 0, all_positions=True)
    for b in range(TOY.B):
        ref = np.array(scalar_forward(TOY, W, toks[b].tolist()))
        # a bf16 rounding can flip when the two summation orders differ in the last fp32 bit; allow that
        assert np.abs(got[b] - ref).max() < 2e-3 * max(1.0, np.abs(ref).max())
        assert np.mean(np.abs(got[b] - ref)) < 1e-4


def test_prefill_decode_equivalence():
    """Prefill of S+1 tokens gives the same last logits as prefill of S then one decode step."""
    toks = np.concatenate([si.prompt_tokens(TOY), np.array([[3], [17]], dtype=np.int32)], axis=1)
    cfg = replace(TOY, S=6)
    a, _ = toy_model(cfg)
    full = a.step(toks, 0)
    b, _ = toy_model(cfg)
    b.step(toks[:, :5], 0)
    inc = b.step(toks[:, 5:], 5)
    assert np.abs(full - inc).max() < 1e-5


def test_batch_invariance_and_causality():
    m, _ = toy_model()
    toks = si.prompt_tokens(TOY)
    allp = m.step(toks, 0, all_positions=True)
    one = replace(TOY, B=1)
    for b in range(TOY.B):
        m1, _ = toy_model(one)
        assert np.array_equal(m1.step(toks[b:b + 1], 0, all_positions=True)[0], allp[b])
    t2 = toks.copy()
    t2[:, 3:] = (t2[:, 3:] + 7) % TOY.V
    m2, _ = toy_model()
    allp2 = m2.step(t2, 0, all_positions=True)
    assert np.array_equal(allp2[:, :3], allp[:, :3]) and not np.array_equal(allp2[:, 3:], allp[:, 3:])


def test_zero_output_projections_closed_form():
    """With Wo = Wd = 0 the residual stream is the embedding: logits = bf16(rms(embed[tok])) . Wlm."""
    lay = si.build_layout(TOY)
    W = si.weights_as_bits(lay)
    for l in range(TOY.L):
        W[(si.K_WO, l, -1)][:] = 0
        W[(si.K_WD, l, -1)][:] = 0
    m = OracleModel(TOY, W)
    toks = si.prompt_tokens(TOY)
    got = m.step(toks, 0)
    e = si.bf16_bits_to_f32(W[(si.K_EMBED, -1, -1)]).astype(np.float64)[toks[:, -1]]
    h = e / np.sqrt((e * e).mean(-1, keepdims=True) + TOY.eps)
    h = si.bf16_bits_to_f32(si.f32_to_bf16_bits(h.astype(np.float32))).astype(np.float64)
    ref = h @ si.bf16_bits_to_f32(W[(si.K_LM, -1, -1)]).astype(np.float64).T
    assert np.abs(got - ref).max() < 1e-6


def test_rope_properties():
    m, _ = toy_model()
    rng = np.random.default_rng(1)
    t = rng.standard_normal((1, 3, 4, TOY.Dh)).astype(np.float32)
    r0 = m.rope(t[:, :1], 0)
    assert np.array_equal(r0, t[:, :1])                                   # position 0: identity
    r = m.rope(t, 2)
    assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(t, axis=-1), rtol=1e-6)    # rotation
    # relative-position property: <rope(q,p), rope(k,p')> depends on p - p' only
    q, k = t[:, :1, :1], t[:, 1:2, :1]
    d1 = (m.rope(q, 3) * m.rope(k, 1)).sum()
    d2 = (m.rope(q, 5) * m.rope(k, 3)).sum()
    assert abs(d1 - d2) < 1e-5
    c, s = rope_table(8, 4, 10000.0)
    assert c.shape == (4, 4) and np.isclose(c[1, 0], math.cos(1.0)) and np.isclose(s[1, 1], math.sin(10000 ** -0.25))


def test_attention_single_token_returns_v_and_matches_torch_sdpa():
    import torch
    cfg = replace(TOY, B=1)
    m, _ = toy_model(cfg)
    rng = np.random.default_rng(2)
    kv = bf16_round(rng.standard_normal((cfg.Hkv, 6, cfg.Dh)).astype(np.float32))
    vv = bf16_round(rng.standard_normal((cfg.Hkv, 6, cfg.Dh)).astype(np.float32))
    m.K[0, 0, :, :6], m.V[0, 0, :, :6] = kv, vv
    q = bf16_round(rng.standard_normal((1, 1, cfg.Hq, cfg.Dh)).astype(np.float32))
    o = m.attention(0, q, 0)                       # kvlen = 1: softmax over one key
    for h in range(cfg.Hq):
        assert np.array_equal(o[0, 0, h], vv[h // 2, 0])
    qs = bf16_round(rng.standard_normal((1, 6, cfg.Hq, cfg.Dh)).astype(np.float32))
    o = m.attention(0, qs, 0)                      # 6 queries, causal
    tq = torch.from_numpy(qs.astype(np.float64)).permute(0, 2, 1, 3)
    tk = torch.from_numpy(kv.astype(np.float64))[None].repeat_interleave(2, dim=1)
    tv = torch.from_numpy(vv.astype(np.float64))[None].repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(0, 2, 1, 3).numpy()
    assert np.abs(o - ref).max() < 1e-5


def test_linear_is_x_times_w_transposed():
    m, W = toy_model()
    rng = np.random.default_rng(3)
    a = rng.standard_normal((3, TOY.d))
    Wq = si.bf16_bits_to_f32(W[(si.K_WQ, 0, -1)]).astype(np.float64)
    ref = np.array([[sum(a[r, i] * Wq[o, i] for i in range(TOY.d)) for o in range(Wq.shape[0])] for r in range(3)])
    assert np.abs(m.linear(a, m.w[(si.K_WQ, 0, -1)]) - ref).max() < 1e-5


def test_moe_single_expert_equals_dense_and_gates_sum_to_one():
    dense = replace(TOY, L=1)
    moe = replace(TOY, L=1, E=1, topk=1)
    lay = si.build_layout(dense)
    W = si.weights_as_bits(lay)
    Wm = {k: v for k, v in W.items() if k[0] not in (si.K_WG, si.K_WU, si.K_WD)}
    for k in (si.K_WG, si.K_WU, si.K_WD):
        Wm[(k, 0, 0)] = W[(k, 0, -1)]
    Wm[(si.K_ROUTER, 0, -1)] = si.normal_bf16_bits(1, 2, 0, dense.d).reshape(1, dense.d)
    toks = si.prompt_tokens(dense)
    a = OracleModel(dense, W).step(toks, 0)
    b = OracleModel(moe, Wm, np.zeros((1, 1), np.float32)).step(toks, 0)
    assert np.abs(a - b).max() < 1e-6


def test_moe_top2_routing_counts_and_tie_break():
    cfg = replace(TOY, L=1, E=4, topk=2)
    lay = si.build_layout(cfg)
    W = si.weights_as_bits(lay)
    W[(si.K_ROUTER, 0, -1)][:] = 0                  # logits = bias only: every token picks the same two experts
    bias = np.array([[0.5, 1.0, 1.0, -2.0]], dtype=np.float32)      # tie between experts 1 and 2 -> 1 first
    m = OracleModel(cfg, W, bias)
    m.step(si.prompt_tokens(cfg), 0)
    assert m.expert_counts[0][0].tolist() == [0, cfg.B * cfg.S, cfg.B * cfg.S, 0]
    bias2 = np.array([[1.0, 1.0, 1.0, 1.0]], dtype=np.float32)      # four-way tie -> experts 0 and 1
    m2 = OracleModel(cfg, W, bias2)
    m2.step(si.prompt_tokens(cfg), 0)
    assert m2.expert_counts[0][0].tolist() == [cfg.B * cfg.S, cfg.B * cfg.S, 0, 0]


MOE_TOY = replace(TOY, L=2, E=4, topk=2, F=16)


def test_moe_top2_matches_scalar_loops():
    """The whole mixture-of-experts forward pass (router, top-2 with the tie rule, softmax over the two selected logits
    only, gate <-> expert pairing, scaling after the down projection, summation in ascending expert id) against plain
    Python loops in double.  A softmax over all E logits, gates swapped between the two slots, or the gate applied
    before the down projection's fp32 rounding all move the logits by far more than the tolerance."""
    cfg = MOE_TOY
    m, W = toy_model(cfg)
    bias = si.router_bias(cfg)
    toks = si.prompt_tokens(cfg)
    got = m.step(toks, 0, all_positions=True)
    seen = np.zeros((cfg.L, cfg.E), dtype=np.int64)
    for b in range(cfg.B):
        routed = []
        ref = np.array(scalar_forward(cfg, W, toks[b].tolist(), bias, routed))
        assert np.abs(got[b] - ref).max() < 2e-3 * max(1.0, np.abs(ref).max())
        assert np.mean(np.abs(got[b] - ref)) < 1e-4
        for (l, p, choice) in routed:
            assert len(choice) == 2 and abs(sum(g for _, g in choice) - 1.0) < 1e-6
            for e, g in choice:
                seen[l, e] += 1
    assert [c.tolist() for c in m.expert_counts[0]] == seen.tolist()
    assert (seen > 0).sum() >= 5                 # the toy routes to several experts, with unequal gates
    # the same pass with the two gates of every token exchanged must NOT pass: the pin would catch a swapped pairing
    class Swapped(OracleModel):
        def ffn_moe(self, l, h2, x):
            cfg_ = self.cfg
            logits = (h2.astype(np.float64) @ self.w[(self.ROUTER, l, -1)].T + self.bias[l]).astype(np.float32)
            order = np.argsort(-logits, axis=-1, kind="stable")[:, :2]
            sel = np.take_along_axis(logits, order, axis=-1).astype(np.float64)
            ex = np.exp(sel - sel.max(axis=-1, keepdims=True))
            gates = (ex / ex.sum(axis=-1, keepdims=True)).astype(np.float32)[:, ::-1]
            counts = np.zeros(cfg_.E, dtype=np.int64)
            for e in range(cfg_.E):
                rows, slot = np.nonzero(order == e)
                counts[e] = len(rows)
                if len(rows):
                    x[rows] = (x[rows].astype(np.float64) + gates[rows, slot][:, None] * self.ffn_dense(l, h2[rows], e)).astype(np.float32)
            return x, counts
    lay = si.build_layout(cfg)
    bad = Swapped(cfg, W, bias).step(toks, 0, all_positions=True)
    ref0 = np.array(scalar_forward(cfg, W, toks[0].tolist(), bias))
    assert np.abs(bad[0] - ref0).max() > 20 * 2e-3 * max(1.0, np.abs(ref0).max())


def test_moe_gates_closed_forms():
    """Router weights zero, so the logits are the bias.  (1) Two experts with equal logits and equal weights: gates
    1/2, 1/2, and y/2 + y/2 is exactly the dense FFN's y.  (2) Bias (ln 3, 0, -1/2, -1/2) over four experts: the top
    two are experts 0 and 1 with gates 3/4 and 1/4 - a softmax over all four logits would give 0.575 and 0.192 - and
    with expert 1's down projection zeroed the layer adds exactly 3/4 of expert 0's output; with expert 0's zeroed,
    1/4 of expert 1's: the gate goes with its own expert."""
    dense = replace(TOY, L=1)
    lay = si.build_layout(dense)
    W = si.weights_as_bits(lay)
    for k, v in W.items():
        if k[0] not in (si.K_G1, si.K_G2, si.K_GF):
            W[k] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(v) * np.float32(8.0))
    toks = si.prompt_tokens(dense)
    base = {k: v for k, v in W.items() if k[0] not in (si.K_WG, si.K_WU, si.K_WD)}
    base[(si.K_ROUTER, 0, -1)] = np.zeros((2, dense.d), dtype=np.uint16)
    two = dict(base)
    for e in range(2):
        for k in (si.K_WG, si.K_WU, si.K_WD):
            two[(k, 0, e)] = W[(k, 0, -1)]
    a = OracleModel(dense, W).step(toks, 0)
    b = OracleModel(replace(dense, E=2, topk=2), two, np.array([[0.3, 0.3]], np.float32)).step(toks, 0)
    assert np.abs(a - b).max() < 1e-6
    # (2) at the level of the layer function, on a zero residual stream
    cfg4 = replace(dense, E=4, topk=2)
    lay4 = si.build_layout(cfg4)
    W4 = si.weights_as_bits(lay4)
    for k, v in W4.items():
        if k[0] not in (si.K_G1, si.K_G2, si.K_GF):
            W4[k] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(v) * np.float32(8.0))
    W4[(si.K_ROUTER, 0, -1)][:] = 0
    bias = np.array([[math.log(3.0), 0.0, -0.5, -0.5]], dtype=np.float32)
    rng = np.random.default_rng(8)
    h2 = bf16_round(rng.standard_normal((5, dense.d)).astype(np.float32)).astype(np.float64)
    for keep, gate in ((0, 0.75), (1, 0.25)):
        Wk = {k: v.copy() for k, v in W4.items()}
        Wk[(si.K_WD, 0, 1 - keep)][:] = 0
        m = OracleModel(cfg4, Wk, bias)
        y, counts = m.ffn_moe(0, h2, np.zeros((5, dense.d), dtype=np.float32))
        assert counts.tolist() == [5, 5, 0, 0]
        want = gate * m.ffn_dense(0, h2, keep).astype(np.float64)
        assert np.abs(y - want).max() < 1e-6 * max(1.0, np.abs(want).max())
        assert np.abs(want).max() > 1e-3


def test_fp32_and_fp64_oracles_agree_on_config_1_prefill():
    cfg = si.CONFIGS[1]
    lay = si.build_layout(cfg)
    W = si.weights_as_bits(lay)
    toks = si.prompt_tokens(cfg)
    a = OracleModel(cfg, W, dtype=np.float64).step(toks, 0)
    b = OracleModel(cfg, W, dtype=np.float32).step(toks, 0)
    assert np.abs(a - b).max() < 3e-3
    assert a.shape == (cfg.B, cfg.V) and np.isfinite(a).all() and a.std() > 1e-3
