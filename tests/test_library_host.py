"""Host side of the library against the oracle: registry, trace, classification and schedule must be
bit-exact (compared as exported blobs); error paths return codes, never crash.  No GPU needed."""
import ctypes
import os
import re
import struct
from dataclasses import replace

import numpy as np
import pytest

import seeded_inputs as si
from conftest import MACHINE
from oracle import policy, trace, validate
from paper_2609_06172_b200 import binding as tb
from paper_2609_06172_b200 import build as tbuild
from paper_2609_06172_b200.session import Session


@pytest.fixture(scope="module", autouse=True)
def _built():
    tbuild.build()


def pack_trace(ops):
    out = []
    for o in ops:
        out.append(struct.pack("<IQiIQQI", o.step, o.site, o.layer, o.kind, o.flops, o.hbm, len(o.acc)))
        out += [struct.pack("<IIQ", *a) for a in o.acc]
    return b"".join(out)


def oracle_blobs(lay, bits=15, expert_counts=None, budget=None):
    ops, steps = trace.run_trace(lay, expert_counts=expert_counts)
    pl = policy.plan(lay.tensors, ops, steps, policy.Machine(**MACHINE), budget or lay.budget, bits)
    return ops, steps, pl.blobs()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(os.path.dirname(tbuild.INCLUDE), "include", "tgp.h")).read()
    declared = set(re.findall(r"\b(tgp_[a-z_0-9]+)\s*\(", hdr))
    lib = ctypes.CDLL(tbuild.LIB)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(tb.exported_symbols())


@pytest.mark.parametrize("c", [1, 2, 3, 4])
def test_plan_bit_exact_dense_configs(c):
    lay = si.build_layout(si.CONFIGS[c])
    s = Session(lay, MACHINE)
    got = s.plan()
    ops, steps, want = oracle_blobs(lay)
    assert s.ctx.trace_export() == pack_trace(ops)
    for k in want:
        assert got[k] == want[k], k
    s.close()


def synthetic_expert_counts(cfg, rng):
    """Top-2 routing counts with a Zipf-like popularity (counts only; no forward pass involved)."""
    p = np.array([r ** -1.2 for r in range(1, cfg.E + 1)])
    p /= p.sum()
    out = np.zeros((1 + cfg.T, cfg.L, cfg.E), dtype=np.uint32)
    for k in range(1 + cfg.T):
        M = cfg.B * (cfg.S if k == 0 else 1)
        for l in range(cfg.L):
            for _ in range(M):
                e = rng.choice(cfg.E, size=2, replace=False, p=p)
                out[k, l, e] += 1
    return out


def test_plan_bit_exact_moe_reduced_and_full_shape():
    rng = np.random.default_rng(5)
    small = replace(si.CONFIGS[5], L=3, B=4, S=8, T=6, TK=4)
    lay = si.build_layout(small, budget=3 << 30)
    ec = synthetic_expert_counts(small, rng)
    s = Session(lay, MACHINE, router_bias=si.router_bias(small))
    got = s.plan(expert_counts=ec)
    ops, steps, want = oracle_blobs(lay, expert_counts=ec)
    assert s.ctx.trace_export() == pack_trace(ops)
    for k in want:
        assert got[k] == want[k], k
    validate.check(lay.tensors, ops, steps, lay.budget, got)
    s.close()
    # full config-5 shape and budget, every expert hit in every step (the worst case for the link)
    cfg = si.CONFIGS[5]
    lay = si.build_layout(cfg)
    ec = np.zeros((1 + cfg.T, cfg.L, cfg.E), dtype=np.uint32)
    ec[0] = cfg.B * cfg.S * 2 // cfg.E
    ec[1:] = cfg.B * 2 // cfg.E
    s = Session(lay, MACHINE, router_bias=si.router_bias(cfg))
    got = s.plan(expert_counts=ec)
    ops, steps, want = oracle_blobs(lay, expert_counts=ec)
    for k in want:
        assert got[k] == want[k], k
    s.close()


@pytest.mark.parametrize("bits", [0, tb.BIT_A, tb.BIT_P, tb.BIT_A | tb.BIT_P, tb.BIT_ZC, 7, tb.BIT_W, 15])
def test_plan_bit_exact_under_ablation_bits(bits):
    lay = si.build_layout(si.CONFIGS[1])
    s = Session(lay, MACHINE)
    try:
        got = s.plan(bits=bits)
    except tb.TgpError as e:
        assert e.code == tb.E_BUDGET_TOO_SMALL
        with pytest.raises(policy.PlanError):
            oracle_blobs(lay, bits)
        return
    ops, steps, want = oracle_blobs(lay, bits)
    for k in want:
        assert got[k] == want[k], (bits, k)
    validate.check(lay.tensors, ops, steps, lay.budget, got)
    s.close()


@pytest.mark.parametrize("first_step", [0, 2, 20])
def test_windowed_pin_reservation_is_bit_exact_and_moves_fewer_bytes(first_step):
    """A long decode on a small model whose KV tiles (32 KiB) hold two 16 KiB weight blocks: the slots of the tiles born
    in later decode steps house unpinned weight blocks until then.  Library and oracle agree bit for bit, with the bit
    on and off, for the whole run and for a tail plan; the windowed plan passes the validator and moves fewer bytes."""
    cfg = replace(si.CONFIGS[1], B=4, S=30, T=40, TK=16)
    lay = si.build_layout(cfg, cap=16 << 10)
    ops, steps = trace.run_trace(lay)
    mach = policy.Machine(**MACHINE)
    totals = {}
    for bits in (7, 15):
        s = Session(lay, MACHINE)
        got = s.plan(bits=bits)
        if first_step:
            s.ctx.replan_begin(first_step)
            s.ctx.replan_wait()
            got = s.ctx.plan_blobs(tail=True)
            want = policy.plan_tail(lay.tensors, ops, steps, mach, lay.budget, first_step, bits=bits).blobs()
        else:
            want = policy.plan(lay.tensors, ops, steps, mach, lay.budget, bits=bits).blobs()
        for k in want:
            assert got[k] == want[k], (bits, k)
        validate.check(lay.tensors, ops, steps, lay.budget, got, first_step=first_step)
        totals[bits] = int(np.frombuffer(got["totals"], dtype="<u8").reshape(-1, 4)[:, 0].sum())
        s.close()
    if first_step == 0:
        assert totals[15] < totals[7]
    else:
        assert totals[15] <= totals[7]


def test_library_plan_passes_the_validator_config_2():
    lay = si.build_layout(si.CONFIGS[2])
    s = Session(lay, MACHINE)
    got = s.plan(T=8)
    ops, steps = trace.run_trace(lay, n_decode=8)
    validate.check(lay.tensors, ops, steps, lay.budget, got)
    s.close()


def test_schedule_is_independent_of_the_pool_address():
    lay = si.build_layout(si.CONFIGS[1])
    a = Session(lay, MACHINE, pool_base=1 << 30)
    b = Session(lay, MACHINE, pool_base=(7 << 40) + 512 * 12345)
    assert a.plan() == b.plan()
    assert a.ctx.tensor_identity(17) == b.ctx.tensor_identity(17)
    a.close(), b.close()


def test_trace_recorded_through_the_c_calls_equals_model_trace():
    lay = si.build_layout(si.CONFIGS[1])
    ops, steps = trace.run_trace(lay, n_decode=2)
    s = Session(lay, MACHINE)
    s.ctx.trace_begin()
    for (kind, first, count) in steps:
        s.ctx.trace_step(kind)
        for o in ops[first:first + count]:
            s.ctx.trace_op(o.site, o.layer, o.kind, o.flops, o.hbm, o.acc)
    s.ctx.trace_end()
    s.ctx.plan()
    manual = s.ctx.plan_blobs()
    assert s.plan(T=2) == manual
    s.close()


def test_registry_lookup_identity_and_errors():
    ctx = tb.Ctx(**MACHINE)
    buf = np.zeros(1 << 16, dtype=np.uint8)
    base = (buf.ctypes.data + 511) // 512 * 512
    pool = ctx.pool_register(base, 32768, tb.POOL_PLAIN)
    a = ctx.tensor_register(pool, 0, 1000, 0xABC, 0, 2, tb.T_READONLY)
    b = ctx.tensor_register(pool, 4096, 2048, 0xABC, 0, 3, tb.T_READONLY)
    c = ctx.tensor_register(pool, 1024, 512, 0xDEF, 1, 13, tb.T_MUTABLE)       # out of address order
    assert ctx.tensor_lookup(base + 999) == (a, 999)
    assert ctx.tensor_lookup(base + 4096 + 7) == (b, 7)
    assert ctx.tensor_lookup(base + 1024) == (c, 0)
    assert ctx.tensor_identity(a) == (0xABC, 0) and ctx.tensor_identity(b) == (0xABC, 1) and ctx.tensor_identity(c) == (0xDEF, 0)
    for args, code in [((pool, 512, 1024, 1, 0, 2, tb.T_READONLY), tb.E_OVERLAP),        # into a and c
                       ((pool, 3584, 1024, 1, 0, 2, tb.T_READONLY), tb.E_OVERLAP),       # into b
                       ((pool, 32768 - 512, 1024, 1, 0, 2, tb.T_READONLY), tb.E_RANGE),
                       ((pool, 100, 8, 1, 0, 2, tb.T_READONLY), tb.E_INVAL),             # unaligned
                       ((pool + 5, 0, 8, 1, 0, 2, tb.T_READONLY), tb.E_INVAL),
                       ((pool, 8192, 8, 1, 0, 2, 3), tb.E_INVAL)]:
        with pytest.raises(tb.TgpError) as ei:
            ctx.tensor_register(*args)
        assert ei.value.code == code
    for addr in (base + 1000, base + 3000, base - 1, base + 40000):
        with pytest.raises(tb.TgpError) as ei:
            ctx.tensor_lookup(addr)
        assert ei.value.code == tb.E_RANGE
    with pytest.raises(tb.TgpError) as ei:
        ctx.pool_register(base + 512, 1024, tb.POOL_PLAIN)
    assert ei.value.code == tb.E_OVERLAP
    # trace errors
    with pytest.raises(tb.TgpError):
        ctx.plan()                                               # nothing traced
    ctx.trace_begin()
    ctx.trace_step(tb.PREFILL)
    for acc, code in [([(99, tb.R, 8)], tb.E_UNKNOWN_TENSOR), ([(a, tb.W, 8)], tb.E_INVAL), ([(a, tb.R, 8), (a, tb.R, 8)], tb.E_INVAL)]:
        with pytest.raises(tb.TgpError) as ei:
            ctx.trace_op(1, 0, 2, 10, 10, acc)
        assert ei.value.code == code
    ctx.trace_op(1, 0, 2, 10, 10, [(a, tb.R, 1000)])
    ctx.trace_end()
    with pytest.raises(tb.TgpError) as ei:
        ctx.plan()                                               # no budget
    assert ei.value.code == tb.E_STATE
    ctx.set_budget(1024)
    with pytest.raises(tb.TgpError) as ei:
        ctx.plan()
    assert ei.value.code == tb.E_BUDGET_TOO_SMALL
    with pytest.raises(tb.TgpError) as ei:
        ctx.plan_export(tb.X_COMMANDS)
    assert ei.value.code == tb.E_NO_PLAN
    ctx.set_budget(4096)
    ctx.plan()
    assert len(ctx.plan_export(tb.X_COMMANDS)) == 45
    with pytest.raises(tb.TgpError):
        ctx.tensor_register(pool, 16384, 512, 1, 0, 2, tb.T_READONLY)     # registry frozen after tracing
    # stepping without a device binding is a state error, not a crash
    with pytest.raises(tb.TgpError) as ei:
        ctx.step(tb.PREFILL, np.zeros(4, np.int32), 1, 4, 1 << 20, None, None, None)
    assert ei.value.code == tb.E_STATE
    ctx.close()


def test_model_bind_rejects_bad_shapes_and_roles():
    lay = si.build_layout(si.CONFIGS[1])
    s = Session(lay, MACHINE)
    bad = tb.ModelCfg(4, 256, 4, 3, 64, 1024, 4096, 0, 0, 1, 48, 16, 10000.0, 1e-5)          # Hq % Hkv != 0
    with pytest.raises(tb.TgpError):
        s.ctx.model_bind(bad, s.roles)
    long_ctx = tb.ModelCfg(4, 256, 4, 4, 64, 1024, 4096, 0, 0, 1, 65 * 16, 16, 10000.0, 1e-5)   # 65 tiles > 64
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.model_bind(long_ctx, s.roles)
    assert ei.value.code == tb.E_TOO_LARGE
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.model_bind(s.cfg, s.roles + [s.roles[0]])
    assert ei.value.code == tb.E_INVAL
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.model_trace(40, 16)                                # S + T beyond max_len
    assert ei.value.code == tb.E_INVAL
    s.close()


def test_step_refuses_host_tokens_outside_the_vocabulary_before_touching_a_device():
    """A host token id outside [0, V) would send the embedding gather past its table; tgp_step() must refuse it at the
    boundary (no GPU involved: the check comes before the engine is looked at), and an op whose tensor has no model role
    must be a mismatch code, not a crash."""
    lay = si.build_layout(si.CONFIGS[1])
    s = Session(lay, MACHINE)
    s.plan(T=1)
    cfg = lay.cfg
    dummy = np.zeros(16, dtype=np.float32)                      # stands for the logits pointer; never written without a workspace
    for bad in (-1, cfg.V, 2 ** 31 - 1):
        tok = np.zeros((cfg.B, cfg.S), dtype=np.int32)
        tok[0, 5] = bad
        with pytest.raises(tb.TgpError) as ei:
            s.ctx.step(tb.PREFILL, tok, cfg.B, cfg.S, dummy, None, None, None)
        assert ei.value.code == tb.E_INVAL and "vocabulary" in str(ei.value)
    ok = np.full((cfg.B, cfg.S), cfg.V - 1, dtype=np.int32)
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.step(tb.PREFILL, ok, cfg.B, cfg.S, dummy, None, None, None)
    assert ei.value.code == tb.E_STATE                          # legal tokens get as far as "no workspace bound"
    s.close()


def test_replan_from_a_timing_log_is_bit_exact_and_changes_classes():
    """Runtime monitor: the same integer log of kernel times fed to both planners gives the same schedule; an op whose
    kernel ran longer than its bytes take on the link stops being link-bound, and its tensors lose their pin score."""
    lay = si.build_layout(si.CONFIGS[1])
    ops, steps = trace.run_trace(lay)
    rng = np.random.default_rng(11)
    # synthetic log: most ops fast (1 us), a third not measured (0), norm ops slow (20 us >> 512 B over the link)
    ns = np.where(rng.random(len(ops)) < 0.33, 0, 1000).astype(np.uint64)
    for i, o in enumerate(ops):
        if o.kind == trace.OP_RMSNORM:
            ns[i] = 20000
    s = Session(lay, MACHINE)
    base = s.plan()
    s.ctx.set_measured_times(ns)
    s.ctx.plan()
    got = s.ctx.plan_blobs()
    want = policy.plan(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget, measured_ns=ns.tolist()).blobs()
    assert got == want
    validate.check(lay.tensors, ops, steps, lay.budget, got)
    assert got["classes"] != base["classes"]
    norm_ops = [i for i, o in enumerate(ops) if o.kind == trace.OP_RMSNORM]
    assert all(base["classes"][i] == policy.CLS_LINK for i in norm_ops) and all(got["classes"][i] != policy.CLS_LINK for i in norm_ops)
    gain = lay.blocks(si.K_G1, 0)[0].tid
    crit = lambda blobs, t: blobs["tensors"][t * 10]
    assert crit(base, gain) == 1 and crit(got, gain) == 0
    # clearing the log restores the analytic plan; a log of the wrong length is refused
    s.ctx.set_measured_times(None)
    s.ctx.plan()
    assert s.ctx.plan_blobs() == base
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.set_measured_times(ns[:-1])
    assert ei.value.code == tb.E_STATE
    s.close()


@pytest.mark.parametrize("c,first_step", [(1, 1), (1, 9), (2, 3)])
def test_tail_replan_in_the_middle_of_a_run_is_bit_exact(c, first_step):
    """Runtime monitor, second half: the steps from a boundary on are planned again, as a trace of their own, from the
    timing log so far, on a helper thread.  The same integer log fed to the oracle's tail planner gives the same blobs;
    the tail plan passes the validator started from an empty arena with the earlier steps' writes in the pool."""
    cfg = si.CONFIGS[c] if c == 1 else replace(si.CONFIGS[c], T=6)
    lay = si.build_layout(cfg)
    ops, steps = trace.run_trace(lay)
    first_op = steps[first_step][1]
    rng = np.random.default_rng(first_step)
    ns = np.zeros(len(ops), dtype=np.uint64)
    ns[:first_op] = rng.integers(500, 40000, first_op)                    # measured so far
    # ops still to come: the time of the same op in the last measured step of the same kind, where there is one
    if first_step >= 2:
        o0, n = steps[first_step - 1][1], steps[first_step - 1][2]
        for k in range(first_step, len(steps)):
            if steps[k][2] == n:
                ns[steps[k][1]: steps[k][1] + n] = ns[o0: o0 + n]
    s = Session(lay, MACHINE)
    base = s.plan(T=cfg.T)
    s.ctx.replan_begin(first_step, ns)
    s.ctx.replan_wait()
    got = s.ctx.plan_blobs(tail=True)
    assert s.ctx.plan_blobs() == base                                     # the plan in use is untouched until the commit
    want = policy.plan_tail(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget, first_step, measured_ns=ns.tolist()).blobs()
    assert got == want
    validate.check(lay.tensors, ops, steps, lay.budget, got, first_step=first_step)
    assert len(got["classes"]) == len(ops) - first_op and len(got["totals"]) == 32 * (len(steps) - first_step)
    # without a log the tail plan is the analytic one
    s.ctx.set_measured_times(None)
    s.ctx.plan()
    s.ctx.replan_begin(first_step)
    s.ctx.replan_wait()
    assert s.ctx.plan_blobs(tail=True) == policy.plan_tail(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget, first_step).blobs()
    # call-order and argument errors are codes
    for bad in (0, len(steps)):
        with pytest.raises(tb.TgpError) as ei:
            s.ctx.replan_begin(bad)
        assert ei.value.code == tb.E_INVAL
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.replan_begin(first_step, ns[:-1])
    assert ei.value.code == tb.E_INVAL
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.replan_commit()                                             # no engine without a device
    assert ei.value.code == tb.E_STATE
    s.close()


def _resident_of(blobs, n_tensors, first_op):
    """tensor -> arena offset of the pins of a plan that are on the device when op first_op starts: placed before it, or
    never placed at all (kept by that plan itself)."""
    P = validate.parse(blobs, n_tensors)
    placed = {}
    for (seq, kind, t, nb, po, ao, w, f, r) in P["cmds"]:
        if kind != validate.CMD_D2H:
            placed.setdefault((t, ao), f)
    return {t: o for t, o in P["pins"] if placed.get((t, o), -1) < first_op}


@pytest.mark.parametrize("c,first_step", [(1, 2), (1, 9), (2, 3)])
def test_tail_replan_that_keeps_the_resident_pins_is_bit_exact(c, first_step):
    """With tgp_set_replan_keep the tail plan keeps the pinned tensors that are on the device at the boundary: same blobs as
    the oracle's tail planner given that resident set, valid for a replay that starts with them resident, nothing of
    them placed again, fewer bytes in the first tail step than a tail that starts cold; with the switch off again the
    planner returns the cold tail."""
    cfg = si.CONFIGS[c] if c == 1 else replace(si.CONFIGS[c], T=8)
    lay = si.build_layout(cfg)
    ops, steps = trace.run_trace(lay)
    mach = policy.Machine(**MACHINE)
    rng = np.random.default_rng(10 + first_step)
    ns = np.zeros(len(ops), dtype=np.uint64)
    ns[:steps[first_step][1]] = rng.integers(500, 40000, steps[first_step][1])
    s = Session(lay, MACHINE)
    base = s.plan(T=cfg.T)
    s.ctx.replan_begin(first_step, ns)
    s.ctx.replan_wait()
    cold = s.ctx.plan_blobs(tail=True)
    s.ctx.set_replan_keep(True)
    s.ctx.replan_begin(first_step, ns)
    s.ctx.replan_wait()
    got = s.ctx.plan_blobs(tail=True)
    res = _resident_of(base, len(lay.tensors), steps[first_step][1])
    assert res
    want = policy.plan_tail(lay.tensors, ops, steps, mach, lay.budget, first_step, measured_ns=ns.tolist(), resident=res).blobs()
    assert got == want
    validate.check(lay.tensors, ops, steps, lay.budget, got, first_step=first_step, resident=res)
    P = validate.parse(got, len(lay.tensors))
    off = dict(P["pins"])
    kept = {t for t, o in res.items() if off.get(t) == o}
    assert kept and not ({c[2] for c in P["cmds"] if c[1] != validate.CMD_D2H} & kept)
    assert validate.parse(got, len(lay.tensors))["totals"][0][0] < validate.parse(cold, len(lay.tensors))["totals"][0][0]
    s.ctx.set_replan_keep(False)
    s.ctx.replan_begin(first_step, ns)
    s.ctx.replan_wait()
    assert s.ctx.plan_blobs(tail=True) == cold                              # the switch is per plan: off again, the cold tail again
    s.close()


def test_measured_time_link_test_by_hand():
    toy = policy.Machine(1000, 100, 10, 10)            # link 10 B/s
    # 100 bytes over the link take 10 s: a 9 s kernel is link-bound, a 10 s or 11 s kernel is not
    assert policy.classify(5000, 300, 100, toy, measured_ns=9_000_000_000) == policy.CLS_LINK
    assert policy.classify(5000, 300, 100, toy, measured_ns=10_000_000_000) == policy.CLS_COMPUTE
    assert policy.classify(100, 600, 100, toy, measured_ns=11_000_000_000) == policy.CLS_HBM
    assert policy.classify(5000, 300, 100, toy, measured_ns=0) == policy.CLS_LINK          # no measurement: analytic


def test_aliased_host_pool_shares_pages_between_layer_groups_only():
    """The fallback for pools larger than the host can page-lock: layers l and l + phys share physical pages, everything
    else (embedding, head, KV tiles) stays private, and the virtual layout is the ordinary one."""
    from paper_2609_06172_b200.runner import AliasedPool
    cfg = replace(si.CONFIGS[1], L=6, d=1024, F=4096, Hq=16, Hkv=16)   # layer regions are multiples of the page size here
    lay = si.build_layout(cfg)
    try:
        p = AliasedPool(lay, 2)
    except ValueError as ex:
        pytest.skip(f"layout not page-aligned on this machine: {ex}")
    a = p.numpy()
    assert a.size == lay.pool_bytes and p.phys_bytes - lay.pool_bytes + 4 * p.layer_bytes in range(0, 4096)      # fresh pages read as zero
    w = [t for t in lay.tensors if t.kind == si.K_WQ]
    by_layer = {t.layer: t for t in w}
    a[by_layer[1].pool_off] = 7                                     # layer 1 ...
    assert a[by_layer[3].pool_off] == 7 and a[by_layer[5].pool_off] == 7        # ... is layers 3 and 5
    assert a[by_layer[0].pool_off] == 0 and a[by_layer[2].pool_off] == 0
    kv = [t for t in lay.tensors if t.kind == si.K_KT]
    a[kv[0].pool_off] = 9
    assert sum(int(a[t.pool_off] == 9) for t in kv) == 1            # KV tiles are private
    emb = next(t for t in lay.tensors if t.kind == si.K_EMBED)
    a[emb.pool_off + 5] = 3
    assert int((a[:emb.size] == 3).sum()) == 1 and all(int(a[t.pool_off + 5]) != 3 for t in w)
    p.close()
