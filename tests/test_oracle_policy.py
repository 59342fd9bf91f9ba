"""Pins for the oracle trace and policy: hand-computed toy rooflines and op counts, an independent
validator (with mutation tests proving it rejects broken plans), closed forms and a brute-force
search over pin sets."""
import itertools
import os
import struct
from dataclasses import dataclass, replace

import pytest

import seeded_inputs as si
from oracle import policy, trace, validate
from conftest import MACHINE

M = policy.Machine(**MACHINE)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_toy_rooflines_from_fixture():
    toy = policy.Machine(1000, 100, 10, 10)
    names = {"LINK": policy.CLS_LINK, "HBM": policy.CLS_HBM, "COMPUTE": policy.CLS_COMPUTE}
    n = 0
    for line in open(os.path.join(GOLD, "toy_roofline.txt")):
        line = line.split("#")[0].split()
        if len(line) == 4:
            f, h, g, want = int(line[0]), int(line[1]), int(line[2]), names[line[3]]
            assert policy.classify(f, h, g, toy) == want, line
            n += 1
    assert n >= 8
    assert policy.classify(20000, 300, 100, toy, bit_p=False) == policy.CLS_LINK      # selectivity off


def test_gemm_ridge_on_the_measured_machine():
    """A weight block streamed over the link is LINK-bound iff M < P/Bl (about 24.5k tokens here)."""
    K = n = 8192
    def cls(m):
        return policy.classify(2 * m * K * n, 2 * m * K + 2 * K * n + 4 * m * n, 2 * K * n, M)
    ridge = M.peak_flops // M.h2d_Bps
    assert 24000 < ridge < 25000
    assert cls(1) == policy.CLS_LINK and cls(16384) == policy.CLS_LINK
    assert cls(ridge) == policy.CLS_LINK and cls(ridge + 1) == policy.CLS_COMPUTE and cls(32768) == policy.CLS_COMPUTE


def test_trace_counts_by_hand_config_1():
    # with the recipe's own 512 KiB blocks every FFN matrix is one block and the head four: 55 ops per decode step
    lay = si.build_layout(si.CONFIGS[1])
    ops, steps = trace.run_trace(lay)
    assert steps[1][2] == 1 + 4 * (1 + 3 + 1 + 1 + 1 + 1 + 1 + 1 + 1 + 1) + 1 + 4 + 1
    # the hand computation below is for 128 KiB blocks (four blocks per FFN matrix, sixteen for the head)
    lay = si.build_layout(si.CONFIGS[1], cap=128 << 10)
    ops, steps = trace.run_trace(lay)
    assert len(steps) == 17 and steps[0][0] == trace.STEP_PREFILL and steps[1][0] == trace.STEP_DECODE
    pre = ops[steps[0][1]: steps[0][1] + steps[0][2]]
    dec = ops[steps[1][1]: steps[1][1] + steps[1][2]]
    # embed gather, prefill: 32 tokens x 256 x (2 read + 4 written)
    assert (pre[0].kind, pre[0].flops, pre[0].hbm, pre[0].acc[0][2]) == (trace.OP_EMBED, 0, 32 * 256 * 6, 32 * 256 * 2)
    # decode wq block: M=1, K=256, n=256
    g = [o for o in dec if o.kind == trace.OP_GEMM][0]
    assert (g.flops, g.hbm, g.acc[0][2]) == (131072, 512 + 131072 + 1024, 131072)
    # prefill attention: 4*B*Hq*Dh * S(S+1)/2 = 1024 * 528
    a = [o for o in pre if o.kind == trace.OP_ATTN][0]
    assert a.flops == 540672 and a.hbm == 4 * 32 * 4 * 64 + 4 * 1 * 4 * 32 * 64
    assert [x[2] for x in a.acc] == [8192, 8192, 8192, 8192]          # 2 full K tiles then 2 full V tiles
    # first decode step: position 32 opens tile 2 with one token; attention reads 3 K tiles then 3 V tiles
    r = [o for o in dec if o.kind == trace.OP_ROPE_KV][0]
    assert [(x[1], x[2]) for x in r.acc] == [(trace.MODE_W, 512), (trace.MODE_W, 512)]
    a = [o for o in dec if o.kind == trace.OP_ATTN][0]
    assert a.flops == 4 * 4 * 64 * 33 and [x[2] for x in a.acc] == [8192, 8192, 512] * 2
    # ops per decode step: embed + L*(norm, q,k,v, rope, attn, o, norm, 4 gate, 4 up, swiglu, 4 down) + norm + 16 lm + argmax
    assert len(dec) == 1 + 4 * (1 + 3 + 1 + 1 + 1 + 1 + 4 + 4 + 1 + 4) + 1 + 16 + 1
    # down-projection block carries the residual read: K=1024, n=64
    d = [o for o in dec if o.kind == trace.OP_GEMM and o.site == trace.site_of(trace.OP_GEMM, trace.K_WD)][0]
    assert d.hbm == 2 * 1024 + 2 * 1024 * 64 + 4 * 64 + 4 * 64
    # total flops of a decode step ~ 2 * (params without embed) + attention
    params = (lay.weight_bytes // 2) - 4096 * 256 - 9 * 256
    total = sum(o.flops for o in dec if o.kind == trace.OP_GEMM)
    assert total == 2 * params


def test_moe_trace_lists_only_routed_experts():
    cfg = replace(si.CONFIGS[5], L=2, B=2, S=4, T=1, TK=4)
    lay = si.build_layout(cfg, budget=8 << 30)
    counts = [[[8, 0, 0, 8, 0, 0, 0, 0], [0, 16, 0, 0, 0, 0, 0, 0]], [[2, 2, 0, 0, 0, 0, 0, 0], [0, 0, 0, 0, 0, 0, 1, 3]]]
    ops, steps = trace.run_trace(lay, expert_counts=counts)
    experts = lambda k, l: sorted({o.expert for o in ops[steps[k][1]: steps[k][1] + steps[k][2]] if o.layer == l and o.expert >= 0})
    assert experts(0, 0) == [0, 3] and experts(0, 1) == [1] and experts(1, 1) == [6, 7]
    g = [o for o in ops if o.expert == 7 and o.kind == trace.OP_GEMM][0]
    assert g.m == 3 and g.flops == 2 * 3 * g.acc[0][2] // 2


@pytest.mark.parametrize("c", [1, 2, 3])
def test_plan_invariants(c):
    lay = si.build_layout(si.CONFIGS[c])
    ops, steps = trace.run_trace(lay)
    pl = policy.plan(lay.tensors, ops, steps, M, lay.budget)
    r = validate.check(lay.tensors, ops, steps, lay.budget, pl.blobs())
    assert r["n_cmds"] == len(pl.cmds) and r["n_pins"] == len(pl.pins)
    # every decode op is link-bound or has no pool traffic; the embedding table is read in place
    assert pl.zc[lay.blocks(si.K_EMBED)[0].tid] == 1
    # steady decode step: bytes over the link = accessed non-ZC bytes - pinned accessed bytes
    pinned = {t for t, _ in pl.pins}
    k = len(steps) - 1
    acc = {}
    for o in ops[steps[k][1]: steps[k][1] + steps[k][2]]:
        for (t, mode, touched) in o.acc:
            acc[t] = 1
    want = sum(lay.tensors[t].size for t in acc if t not in pinned and not pl.zc[t])
    assert pl.totals[k][0] == want
    # the policy's own lower bound: a step cannot move less than accessed - budget
    assert pl.totals[k][0] >= sum(lay.tensors[t].size for t in acc if not pl.zc[t]) - lay.budget


def _tamper(blobs, fn):
    rec = struct.Struct("<IBIQQQiii")
    cmds = [list(rec.unpack_from(blobs["commands"], k)) for k in range(0, len(blobs["commands"]), rec.size)]
    fn(cmds)
    out = dict(blobs)
    out["commands"] = b"".join(rec.pack(*c) for c in cmds)
    return out


def test_validator_rejects_broken_plans():
    lay = si.build_layout(si.CONFIGS[1])
    ops, steps = trace.run_trace(lay)
    pl = policy.plan(lay.tensors, ops, steps, M, lay.budget)
    good = pl.blobs()
    validate.check(lay.tensors, ops, steps, lay.budget, good)
    ring = [k for k, c in enumerate(pl.cmds) if c.kind == policy.CMD_H2D and c.arena_off >= pl.ring_base]
    late = ring[len(ring) // 2]

    def drop(cmds):                      # a tensor never staged
        del cmds[late]
        for k, c in enumerate(cmds):
            c[0] = k
    def early(cmds):                     # reuse of ring space before its previous user is done
        for k in ring[20:]:
            cmds[k][6] = -1
    def collide(cmds):                   # two live stays on the same bytes
        cmds[late][5] = cmds[late - 1][5]
    def swap(cmds):                      # order differs from first use
        cmds[late], cmds[late + 8] = cmds[late + 8], cmds[late]
        for k, c in enumerate(cmds):
            c[0] = k
    def outside(cmds):
        cmds[late][5] = lay.budget
    def no_writeback(cmds):
        k = next(k for k, c in enumerate(cmds) if c[1] == policy.CMD_D2H)
        del cmds[k]
        for j, c in enumerate(cmds):
            c[0] = j
    for fn in (drop, early, collide, swap, outside):
        with pytest.raises(validate.PlanInvalid):
            validate.check(lay.tensors, ops, steps, lay.budget, _tamper(good, fn))
    lay2 = si.build_layout(si.CONFIGS[2])
    ops2, steps2 = trace.run_trace(lay2, n_decode=4)
    pl2 = policy.plan(lay2.tensors, ops2, steps2, M, lay2.budget, bits=policy.BIT_P | policy.BIT_ZC)     # no pins: KV tiles stream
    assert any(c.kind == policy.CMD_D2H for c in pl2.cmds)
    validate.check(lay2.tensors, ops2, steps2, lay2.budget, pl2.blobs())
    with pytest.raises(validate.PlanInvalid):
        validate.check(lay2.tensors, ops2, steps2, lay2.budget, _tamper(pl2.blobs(), no_writeback))


def test_closed_forms_large_and_minimal_budget():
    lay = si.build_layout(si.CONFIGS[1])
    ops, steps = trace.run_trace(lay)
    accessed = {}
    for o in ops:
        for (t, _, _) in o.acc:
            accessed[t] = lay.tensors[t]
    # (a) budget >= footprint + ring minimum: everything that is read gets exactly one H2D, ever
    big = policy.plan(lay.tensors, ops, steps, M, 4 * lay.pool_bytes)
    h2d = [c for c in big.cmds if c.kind == policy.CMD_H2D]
    assert len({c.tensor for c in h2d}) == len(h2d)
    ro = [t for t in accessed.values() if t.flags == si.F_READONLY and not big.zc[t.tid]]
    assert sum(c.nbytes for c in h2d) == sum(t.size for t in ro)        # KV tiles are born on the device (ALLOC)
    assert not any(c.kind == policy.CMD_D2H for c in big.cmds)
    # (b) no affinity bit: no pins, each step moves every accessed non-ZC byte
    t_only = policy.plan(lay.tensors, ops, steps, M, lay.budget, bits=policy.BIT_P | policy.BIT_ZC)
    assert t_only.pins == [] and t_only.ring_base == 0
    validate.check(lay.tensors, ops, steps, lay.budget, t_only.blobs())
    k = len(steps) - 1
    step_acc = {t for o in ops[steps[k][1]: steps[k][1] + steps[k][2]] for (t, _, _) in o.acc}
    assert t_only.totals[k][0] == sum(lay.tensors[t].size for t in step_acc if not t_only.zc[t])
    # (c) budget below the ring minimum is an error, not a bad plan
    with pytest.raises(policy.PlanError):
        policy.plan(lay.tensors, ops, steps, M, 128 << 10)
    # (d) without zero-copy the embedding table is staged like any tensor
    nozc = policy.plan(lay.tensors, ops, steps, M, lay.budget, bits=policy.BIT_A | policy.BIT_P)
    assert sum(nozc.zc) == 0
    validate.check(lay.tensors, ops, steps, lay.budget, nozc.blobs())


@dataclass
class _T:
    size: int
    pool_off: int
    flags: int = 1


@dataclass
class _O:
    step: int
    flops: int
    hbm: int
    acc: list


def test_greedy_pins_match_brute_force_on_equal_sizes():
    """<= 10 equal-size read-only tensors with different reuse counts: greedy-by-density is optimal."""
    size = 4096
    reuse = [5, 1, 3, 7, 2, 2, 6, 1, 4, 3]
    tensors = [_T(size, k * size) for k in range(len(reuse))]
    ops = []
    for rnd in range(max(reuse)):
        for t, r in enumerate(reuse):
            if rnd < r:
                ops.append(_O(0, 10, 10, [(t, 1, size)]))
                ops += [_O(0, 10, 10, []) for _ in range(policy.W_AFF + 1)]     # gaps: no hold across uses
    steps = [(0, 0, len(ops))]
    for n_pin in (0, 3, 6):
        budget = 2 * size + n_pin * size
        pl = policy.plan(tensors, ops, steps, M, budget)
        validate.check(tensors, ops, steps, budget, pl.blobs())
        got = pl.totals[0][0]
        best = min(sum(size * (1 if t in sub else reuse[t]) for t in range(len(reuse)))
                   for sub in map(set, itertools.combinations(range(len(reuse)), n_pin)))
        assert len(pl.pins) == n_pin and got == best


def test_hold_window_keeps_short_reuse_in_place():
    size = 8192
    tensors = [_T(size, 0), _T(size, size), _T(size, 2 * size, flags=2)]
    acc = lambda t, m=1: [(t, m, size)]
    ops = [_O(0, 1, 1, acc(0)), _O(0, 1, 1, acc(1)), _O(0, 1, 1, acc(0)),          # reuse within the window
           _O(0, 1, 1, []), _O(0, 1, 1, []), _O(0, 1, 1, []), _O(0, 1, 1, []), _O(0, 1, 1, []),
           _O(0, 1, 1, acc(0)),                                                   # beyond the window: new stay
           _O(0, 1, 1, acc(2, 2)), _O(0, 1, 1, acc(2, 1))]                        # written then read: one stay, one D2H
    pl = policy.plan(tensors, ops, [(0, 0, len(ops))], M, 6 * size, bits=policy.BIT_P)
    kinds = [(c.kind, c.tensor, c.first_use, c.release_after) for c in pl.cmds]
    assert kinds == [(policy.CMD_H2D, 0, 0, 2), (policy.CMD_H2D, 1, 1, 1), (policy.CMD_H2D, 0, 8, 8),
                     (policy.CMD_ALLOC, 2, 9, 10), (policy.CMD_D2H, 2, 10, 10)]
    validate.check(tensors, ops, [(0, 0, len(ops))], 6 * size, pl.blobs())


def test_tail_plan_closed_forms_and_invariants():
    """A plan made at a step boundary for the rest of the run: (1) it passes the validator started from an empty arena;
    (2) a KV tile written before the boundary is loaded (H2D), never allocated, at its first access in the tail - a
    tile first written after the boundary is still born on the device; (3) with nothing measured, classes of the tail
    equal the whole-run plan's classes for those ops, and a steady decode step of the tail moves the same bytes as the
    same step of the whole-run plan (same pin capacity, same per-step accesses); (4) a boundary at step 0 is the
    whole-run plan itself."""
    cfg = replace(si.CONFIGS[1], S=30, T=8)             # TK = 16: positions 30, 31 fill tile 1; tile 2 is born at decode step 3
    lay = si.build_layout(cfg)
    ops, steps = trace.run_trace(lay)
    whole = policy.plan(lay.tensors, ops, steps, M, lay.budget)
    assert policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, 0).blobs() == whole.blobs()
    for k in (1, 2, 3, 4, 8):
        tail = policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, k)
        validate.check(lay.tensors, ops, steps, lay.budget, tail.blobs(), first_step=k)
        first_op = steps[k][1]
        assert tail.cls == whole.cls[first_op:]
        written = {t for o in ops[:first_op] for (t, m, _) in o.acc if m & 2}
        later = {t for o in ops[first_op:] for (t, m, _) in o.acc if m & 2} - written
        kinds = {}
        for c in tail.cmds:
            if c.kind != policy.CMD_D2H:
                kinds.setdefault(c.tensor, c.kind)
        assert all(kinds[t] == policy.CMD_H2D for t in written if t in kinds)
        assert all(kinds[t] == policy.CMD_ALLOC for t in later)
        assert (k <= 3) == bool(later)                  # tile 2 of every layer is first written in decode step 3
        assert min(c.first_use for c in tail.cmds) >= first_op and all(c.wait_op == -1 or c.wait_op >= first_op for c in tail.cmds)
        if k <= 6:
            assert tail.totals[-1][0] == whole.totals[-1][0]
    # a tampered tail plan that allocates a tile holding data is caught
    tail = policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, 4)
    blobs = tail.blobs()
    kv = next(c.seq for c in tail.cmds if lay.tensors[c.tensor].flags == si.F_MUTABLE and c.kind == policy.CMD_H2D)
    def to_alloc(cmds):
        cmds[kv][1] = policy.CMD_ALLOC
    with pytest.raises(validate.PlanInvalid):
        validate.check(lay.tensors, ops, steps, lay.budget, _tamper(blobs, to_alloc), first_step=4)


def _resident_at(plan, first_op):
    """tensor -> arena offset of the pins of `plan` that are on the device when op `first_op` starts."""
    off = dict(plan.pins)
    return {c.tensor: c.arena_off for c in plan.cmds if c.kind != policy.CMD_D2H and c.first_use < first_op and off.get(c.tensor) == c.arena_off}


def test_tail_plan_that_keeps_the_resident_pins():
    """A switch of plans in the middle of a run that keeps what is pinned and loaded: (1) the tail plan passes the validator
    started with those tensors resident (a second placement of one of them, or a kept tensor at another offset, is caught);
    (2) with nothing measured the tail pins what the whole-run plan pinned (same densities per step) and every kept pin
    stays at its offset, so the only loads of pinned tensors are those of pins the run had not reached yet; (3) the first
    tail step moves fewer bytes than a tail that starts from an empty arena, by the bytes of the kept pins it touches, and a
    later steady step moves the same; (4) a written KV tile that is kept is never copied from the pool (its copy there is
    stale), one that is not kept is loaded."""
    cfg = replace(si.CONFIGS[1], S=30, T=8)
    lay = si.build_layout(cfg)
    ops, steps = trace.run_trace(lay)
    whole = policy.plan(lay.tensors, ops, steps, M, lay.budget)
    for k in (1, 3, 5):
        first_op = steps[k][1]
        res = _resident_at(whole, first_op)
        assert res
        cold = policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, k)
        keep = policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, k, resident=res)
        validate.check(lay.tensors, ops, steps, lay.budget, keep.blobs(), first_step=k, resident=res)
        with pytest.raises(validate.PlanInvalid):
            validate.check(lay.tensors, ops, steps, lay.budget, keep.blobs(), first_step=k)          # nothing resident: kept pins are missing
        off = dict(keep.pins)
        kept = {t for t, o in res.items() if off.get(t) == o}
        assert kept and all(off[t] == res[t] for t in res if t in off)                              # a resident tensor never moves
        placed = {c.tensor for c in keep.cmds if c.kind != policy.CMD_D2H}
        assert not (placed & kept)
        # pins do not overlap and stay below the ring
        spans = sorted((o, o + policy.alignup(lay.tensors[t].size)) for t, o in keep.pins)
        assert all(b <= c for (a, b), (c, d) in zip(spans, spans[1:])) and spans[-1][1] <= keep.ring_base
        assert keep.ring_base + keep.ring_size == lay.budget
        # bytes: the first tail step saves the kept pins it touches; a steady step costs at most what a cold tail without the
        # windowed reservation costs (the kept plan does not lend late-born pins' slots)
        cold_now = policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, k, bits=policy.BIT_A | policy.BIT_P | policy.BIT_ZC)
        touched = {t for o in ops[first_op:first_op + steps[k][2]] for (t, _, _) in o.acc}
        saved = sum(lay.tensors[t].size for t in kept & touched if t in dict(cold_now.pins))
        assert keep.totals[0][0] <= cold_now.totals[0][0] - saved + sum(lay.tensors[t].size for t in touched if t in dict(cold_now.pins) and t not in off)
        assert keep.totals[0][0] < cold.totals[0][0]
        # written tiles
        written = {t for o in ops[:first_op] for (t, m, _) in o.acc if m & 2}
        assert written & kept
        for c in keep.cmds:
            assert not (c.tensor in kept and c.kind == policy.CMD_H2D)
    # tampering: the same plan with a kept tensor's pin moved is rejected
    k = 3
    first_op = steps[k][1]
    res = _resident_at(whole, first_op)
    keep = policy.plan_tail(lay.tensors, ops, steps, M, lay.budget, k, resident=res)
    moved = dict(res)
    t0 = next(t for t in res if t in dict(keep.pins))
    moved[t0] += 512
    with pytest.raises(validate.PlanInvalid):
        validate.check(lay.tensors, ops, steps, lay.budget, keep.blobs(), first_step=k, resident=moved)


def test_kept_pins_fill_gaps_first_fit_on_a_toy():
    """Hand-checked layout: four read-only tensors of 1, 2, 1 and 1 KiB units are pinned at 0, 1, 3, 4 by the first plan;
    in the tail the second one is no longer used, so a hole of 2 units opens at offset 1.  A tensor of 2 units that the
    tail pins anew goes into that hole (first fit), one of 3 units does not fit any gap below the old end and goes after
    the last kept pin only if the region may grow: the region ends at max(compact size, end of the kept pins)."""
    U = 1024
    sizes = [1 * U, 2 * U, 1 * U, 1 * U, 2 * U, 3 * U]
    tensors = [_T(sz, sum(sizes[:i])) for i, sz in enumerate(sizes)]
    ops, steps = [], []
    def step(st, used):
        o0 = len(ops)
        for t in used:
            ops.append(_O(st, 10, 10, [(t, 1, sizes[t])]))
            ops.extend(_O(st, 10, 10, []) for _ in range(policy.W_AFF + 1))
        steps.append((1 if st else 0, o0, len(ops) - o0))
    step(0, [0, 1, 2, 3]); step(1, [0, 1, 2, 3])
    for st in range(2, 6):
        step(st, [0, 2, 3, 4, 5])
    budget = 2 * 3 * U + 8 * U                       # ring minimum (twice the largest tensor) + room for 8 units of pins
    # (the plan in use was made when only the first two steps were known: it pins tensors 0 - 3, in id order)
    first = policy.plan(tensors, ops[:steps[2][1]], steps[:2], M, budget, bits=policy.BIT_A | policy.BIT_P)
    res = _resident_at(first, steps[2][1])
    assert res == {0: 0, 1: 1 * U, 2: 3 * U, 3: 4 * U}
    tail = policy.plan_tail(tensors, ops, steps, M, budget, 2, bits=policy.BIT_A | policy.BIT_P, resident=res)
    validate.check(tensors, ops, steps, budget, tail.blobs(), first_step=2, resident=res)
    off = dict(tail.pins)
    assert 1 not in off and all(off[t] == res[t] for t in (0, 2, 3))
    hole = res[1]
    assert off[4] == hole                            # two units: exactly the hole the unused tensor left
    end_kept = max(res[t] + sizes[t] for t in (0, 2, 3))
    assert off[5] >= end_kept or 5 not in off        # three units fit no gap between kept pins
    assert tail.ring_base == max(sum(sizes[t] for t in off), end_kept if 5 not in off else off[5] + sizes[5])


def _window_toy(n_w=5, born=3, n_steps=6, size=4096):
    """n_w read-only tensors read once per step, and one mutable tensor of the same size first written in step `born`
    and read and written in every step after it (a KV tile of later positions)."""
    tensors = [_T(size, k * size) for k in range(n_w)] + [_T(size, n_w * size, flags=2)]
    ops, steps = [], []
    for st in range(n_steps):
        o0 = len(ops)
        for t in range(n_w):
            ops.append(_O(st, 10, 10, [(t, 1, size)]))
            ops += [_O(st, 10, 10, []) for _ in range(policy.W_AFF + 1)]
        if st >= born:
            ops.append(_O(st, 10, 10, [(n_w, 2, size)]))
            ops.append(_O(st, 10, 10, [(n_w, 1, size)]))
        steps.append((1 if st else 0, o0, len(ops) - o0))
    return tensors, ops, steps


def test_windowed_reservation_matches_brute_force_on_a_toy_run():
    """The late-born tensor is the densest (a write costs its write-back too), so it is pinned; its slot is idle for the
    first `born` steps.  Static reservation leaves it empty; windowed reservation lends it to the densest unpinned
    tensor, which is then loaded once instead of once per step.  Brute force over every way to use the idle slot (any one
    read-only tensor, or none) gives the same minimum."""
    size = 4096
    for born in (2, 3, 5):
        tensors, ops, steps = _window_toy(born=born, n_steps=born + 4)
        n_w = len(tensors) - 1
        budget = 2 * size + 2 * size                       # ring of two tensors, room for two pins
        static = policy.plan(tensors, ops, steps, M, budget, bits=7)
        windowed = policy.plan(tensors, ops, steps, M, budget, bits=15)
        validate.check(tensors, ops, steps, budget, static.blobs())
        validate.check(tensors, ops, steps, budget, windowed.blobs())
        assert [t for t, _ in static.pins] == [t for t, _ in windowed.pins] and n_w in dict(static.pins)
        h_static = sum(t[0] for t in static.totals)
        h_win = sum(t[0] for t in windowed.totals)
        # by hand: one pinned weight is loaded once, the others every step; the tenant saves (born - 1) loads
        n_steps = len(steps)
        assert h_static == size * (1 + (n_w - 1) * n_steps)
        assert h_win == h_static - size * (born - 1)
        # brute force: the idle slot holds tensor x (or nothing) during steps [0, born)
        pinned_w = [t for t, _ in static.pins if t != n_w][0]
        best = min(h_static - (size * (born - 1) if x is not None else 0) for x in [None] + [t for t in range(n_w) if t != pinned_w])
        assert h_win == best
        # the tenant is the first unpinned tensor in density order (equal densities: lowest id), placed at the landlord's slot
        ten = [c for c in windowed.cmds if c.tensor != n_w and c.tensor not in dict(windowed.pins) and c.arena_off < windowed.ring_base]
        assert len(ten) == 1 and ten[0].arena_off == dict(windowed.pins)[n_w] and ten[0].tensor == min(t for t in range(n_w) if t != pinned_w)
        # the landlord's placement waits for the tenant's last use
        lord = [c for c in windowed.cmds if c.tensor == n_w and c.kind == policy.CMD_ALLOC][0]
        assert lord.wait_op == ten[0].release_after and lord.wait_op < lord.first_use
    # born in step 1: the vacancy is the cold first step only, nothing to save, plans are identical
    tensors, ops, steps = _window_toy(born=1)
    assert policy.plan(tensors, ops, steps, M, 4 * 4096, bits=7).blobs() == policy.plan(tensors, ops, steps, M, 4 * 4096, bits=15).blobs()


def test_validator_rejects_broken_tenancies():
    tensors, ops, steps = _window_toy(born=3)
    budget = 4 * 4096
    pl = policy.plan(tensors, ops, steps, M, budget, bits=15)
    good = pl.blobs()
    validate.check(tensors, ops, steps, budget, good)
    n_w = len(tensors) - 1
    lord = next(c.seq for c in pl.cmds if c.tensor == n_w and c.kind == policy.CMD_ALLOC)
    ten = next(c.seq for c in pl.cmds if c.tensor not in dict(pl.pins) and c.arena_off < pl.ring_base)
    other_pin = next(o for t, o in pl.pins if t != n_w)
    def early_landlord(cmds):                 # the pinned tensor takes its slot while the tenant is still in use
        cmds[lord][6] = -1
    def on_a_resident_pin(cmds):              # a tenant placed over a pinned tensor that is there
        cmds[ten][5] = other_pin
    def overstays(cmds):                      # the tenant claims the slot beyond the landlord's birth
        cmds[ten][8] = cmds[lord][7] + 1
    for fn in (early_landlord, on_a_resident_pin, overstays):
        with pytest.raises(validate.PlanInvalid):
            validate.check(tensors, ops, steps, budget, _tamper(good, fn))
