"""End-to-end parity on the GPU: the planned, oversubscribed forward pass through tgp_step() against the
oracle (teacher-forced tokens), at the tolerance the benchmark spec states: max abs 3e-2, mean relative 1e-2."""
from dataclasses import replace

import numpy as np
import pytest

import seeded_inputs as si
from conftest import MACHINE

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import forward, policy, trace, validate  # noqa: E402
from paper_2609_06172_b200 import binding as tb  # noqa: E402
from paper_2609_06172_b200.runner import Runner, pinned_pool  # noqa: E402
from paper_2609_06172_b200.session import Session  # noqa: E402

MAX_ABS, MEAN_REL = 3e-2, 1e-2          # the tolerance stated for this path


def precision_floor(config):
    """(max abs, mean rel) by which the oracle's own logits move between float32 and float64 accumulation
    (tests/golden/precision_floor.txt, written by make_precision_floor.py from the oracle alone)."""
    import os
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "precision_floor.txt")):
        f = line.split()
        if f and f[0] == str(config):
            return float(f[3]), float(f[5])
    raise KeyError(config)


def setup(cfg, budget=None, bits=15, n_dec=None, cap=None):
    lay = si.build_layout(cfg, budget=budget, cap=cap)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED)
    T = cfg.T if n_dec is None else n_dec
    blobs = s.plan(T=T, bits=bits)
    return lay, pool, s, blobs, T


def check_logits(got, ref, max_abs=MAX_ABS, mean_rel=MEAN_REL):
    worst = 0.0
    for a, b in zip(got, ref):
        err = np.abs(a - b)
        assert err.max() < max_abs, err.max()
        assert err.mean() / np.abs(b).mean() < mean_rel
        worst = max(worst, err.max())
    return worst


def test_config_1_full_run_matches_oracle_and_schedule_is_bit_exact():
    cfg = si.CONFIGS[1]
    lay, pool, s, blobs, T = setup(cfg)
    ops, steps = trace.run_trace(lay)
    want = policy.plan(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget).blobs()
    assert blobs == want
    om = forward.OracleModel(cfg, si.weights_as_bits(lay))
    prompt = si.prompt_tokens(cfg)
    ref, toks = om.generate(prompt, T)
    r = Runner(s, cfg.B * cfg.S)
    got, _ = r.generate(prompt, T, forced=toks)
    assert len(got) == T + 1
    check_logits(got, ref)
    # free-running greedy decode on the device agrees with the oracle's tokens (argmax, lowest id on ties)
    got2, toks2 = r.generate(prompt, T)
    agree = (toks2 == toks).mean()
    assert agree > 0.9, agree
    s.close()


@pytest.mark.parametrize("bits", [0, tb.BIT_A | tb.BIT_P, 7])
def test_oversubscribed_run_is_bitwise_equal_to_a_fully_resident_run(bits):
    """Placement must not change a single bit: 50 % budget (ring + pins, write-backs) vs everything resident."""
    cfg = replace(si.CONFIGS[1], B=2, S=19, T=6, TK=8)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 911 + 3) % cfg.V
    outs = []
    for budget, b in ((None, bits), (64 << 20, 15)):
        lay, pool, s, blobs, T = setup(cfg, budget=budget, bits=b, cap=128 << 10)
        ops, steps = trace.run_trace(lay)
        validate.check(lay.tensors, ops, steps, lay.budget, blobs)
        r = Runner(s, cfg.B * cfg.S)
        got, _ = r.generate(prompt, T, forced=forced)
        outs.append(got)
        if budget is None:
            # KV tiles that were streamed have been written back: host pool holds the device's K/V
            r.sync()
            pins = {t for t, _ in (np.frombuffer(blobs["pins"][:-16], dtype=np.dtype([("t", "<u4"), ("o", "<u8")])).tolist())}
            streamed = [t for t in lay.tensors if t.kind >= si.K_KT and t.tid not in pins]
            if bits == 0:
                assert len(streamed) == len([t for t in lay.tensors if t.kind >= si.K_KT])
            host = pool.numpy()
            nz = sum(int(host[t.pool_off:t.pool_off + t.size].any()) for t in streamed)
            assert nz == len(streamed)
        s.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_ragged_small_model_with_batch_and_gqa():
    cfg = si.ModelConfig("ragged", L=3, d=128, Hq=2, Hkv=1, Dh=64, F=264, V=520, B=3, S=11, T=5, TK=4, seed=5, budget_rule="half_w_kv")
    lay = si.build_layout(cfg, budget=None, cap=16 << 10)
    # weights at std 0.02 and d=128 give tiny logits; scale the test's tolerance check with the reference instead
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED)
    s.plan()
    om = forward.OracleModel(cfg, si.weights_as_bits(lay))
    prompt = si.prompt_tokens(cfg)
    ref, toks = om.generate(prompt, cfg.T)
    r = Runner(s, cfg.B * cfg.S)
    got, _ = r.generate(prompt, cfg.T, forced=toks)
    check_logits(got, ref)
    s.close()


def test_step_stats_and_call_order_errors():
    cfg = si.CONFIGS[1]
    lay, pool, s, blobs, T = setup(cfg, n_dec=2)
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    with pytest.raises(tb.TgpError):
        r.step(tb.DECODE, None, 1)                       # plan starts with a prefill
    st = r.step(tb.PREFILL, prompt, cfg.S, want_stats=True)
    totals = np.frombuffer(blobs["totals"], dtype="<u8").reshape(-1, 4)
    assert (st.h2d_bytes, st.d2h_bytes, st.zc_bytes) == tuple(int(x) for x in totals[0][:3])
    assert st.n_launches > 0 and st.step_ms > 0
    r.step(tb.DECODE, None, 1)
    r.step(tb.DECODE, None, 1)
    with pytest.raises(tb.TgpError) as ei:
        r.step(tb.DECODE, None, 1)                       # plan exhausted
    assert ei.value.code == tb.E_STATE
    r.reset()
    r.step(tb.PREFILL, prompt, cfg.S)
    r.sync()
    s.close()


@pytest.mark.parametrize("budget", [None, 64 << 20])
@pytest.mark.parametrize("B", [1, 2, 5])
def test_decode_step_groups_products_into_one_launch_with_the_same_bits(B, budget):
    """A decode step runs consecutive weight-block products over the same activations (q, k and v; gate and up; the pieces
    of one matrix) as one launch: with everything resident at least two launches fewer per layer; under a budget that
    keeps the ring turning fewer launches too (small blocks whose ring slot a later copy waits for stay alone); not a
    bit of difference in the logits either way; with the switch off every block is its own launch."""
    cfg = replace(si.CONFIGS[1], B=B, S=19, T=5, TK=8)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 577 + 11) % cfg.V
    lay, pool, s, blobs, T = setup(cfg, budget=budget, cap=128 << 10)
    r = Runner(s, cfg.B * cfg.S)
    runs = {}
    for enable in (1, 0):
        tb.k_gemm_group_select(enable)
        logits, launches = [], []
        r.reset()
        r.step(tb.PREFILL, prompt, cfg.S)
        for t in range(T):
            st = r.step(tb.DECODE, np.ascontiguousarray(forced[:, t:t + 1]), 1, want_stats=True)
            launches.append(st.n_launches)
            logits.append(r.logits.cpu().numpy().copy())
        runs[enable] = (logits, launches)
    tb.k_gemm_group_select(1)
    s.close()
    for a, b in zip(runs[1][0], runs[0][0]):
        assert np.array_equal(a, b)
    saved = [u - f for f, u in zip(runs[1][1], runs[0][1])]
    assert min(saved) >= (2 * cfg.L if budget else 1), saved


@pytest.mark.parametrize("B", [1, 2])
def test_decode_step_of_a_small_model_lets_products_compute_their_norm_and_swiglu_with_the_same_bits(B):
    """Launch-bound decode steps: the q/k/v, gate/up and head products normalise the residual stream themselves and the
    down projection computes SwiGLU itself, so those ops launch nothing - fewer launches per step, not a bit of
    difference in any logit (the fused forms redo the separate kernels' arithmetic in the same order)."""
    cfg = replace(si.CONFIGS[1], B=B, S=19, T=6, TK=8)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 577 + 11) % cfg.V
    lay, pool, s, blobs, T = setup(cfg, budget=64 << 20)              # everything resident: every span forms
    r = Runner(s, cfg.B * cfg.S)
    runs = {}
    for enable in (1, 0):
        tb.k_decode_fuse(enable)
        logits, launches = [], []
        r.reset()
        r.step(tb.PREFILL, prompt, cfg.S)
        for t in range(T):
            st = r.step(tb.DECODE, np.ascontiguousarray(forced[:, t:t + 1]), 1, want_stats=True)
            launches.append(st.n_launches)
            logits.append(r.logits.cpu().numpy().copy())
        runs[enable] = (logits, launches)
    tb.k_decode_fuse(0)
    s.close()
    for a, b in zip(runs[1][0], runs[0][0]):
        assert np.array_equal(a, b)
    # per layer two norms and one SwiGLU disappear, and the final norm
    assert all(u - f >= 3 * cfg.L + 1 for f, u in zip(runs[1][1], runs[0][1])), (runs[1][1], runs[0][1])


def test_prefill_swiglu_in_the_up_projection_epilogue_gives_the_same_bits():
    """Prefill of 4 x 200 tokens on a model wide enough for all three tensor-core GEMM kernels (ragged row and column
    tiles): with SwiGLU applied by the up projection's epilogue the step launches one kernel fewer per layer and every
    logit, prefill and the decode steps after it, is bitwise what the separate SwiGLU kernel gives."""
    cfg = replace(si.CONFIGS[1], L=2, d=1024, F=2816, Hq=16, Hkv=4, V=4096, B=4, S=200, T=2, TK=64, budget_rule="half_w")
    lay, pool, s, blobs, T = setup(cfg)
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * T, dtype=np.int32).reshape(cfg.B, T) * 97 + 3) % cfg.V
    runs = {}
    for variant in (0, 1, 2, 3):                                # automatic choice, per-tile, persistent, paired kernel
        for enable in (1, 0):
            tb.k_gemm_tc_variant(variant)
            tb.k_swiglu_epilogue(enable)
            r.reset()
            st = r.step(tb.PREFILL, prompt, cfg.S, want_stats=True)
            logits = [r.logits.cpu().numpy().copy()]
            for t in range(T):
                r.step(tb.DECODE, np.ascontiguousarray(forced[:, t:t + 1]), 1)
                logits.append(r.logits.cpu().numpy().copy())
            runs[(variant, enable)] = (logits, st.n_launches)
    tb.k_gemm_tc_variant(0)
    tb.k_swiglu_epilogue(1)
    assert tb.k_gemm_status() == 0
    s.close()
    for variant in (0, 1, 2, 3):
        on, off = runs[(variant, 1)], runs[(variant, 0)]
        for a, b in zip(on[0], off[0]):
            assert np.array_equal(a, b), variant
        assert off[1] - on[1] == cfg.L
    om = forward.OracleModel(cfg, si.weights_as_bits(lay), dtype=np.float32)
    ref = om.step(prompt, 0)
    check_logits([runs[(0, 1)][0][0]], [ref])


@pytest.mark.parametrize("bits", [tb.BIT_ZC, 15])
def test_adjacent_small_copies_are_coalesced_without_changing_a_bit(bits):
    """Consecutive loads whose pool ranges and arena slots continue one another travel in one copy: with nothing pinned
    (every tensor streamed, neighbours in the pool are neighbours in the ring) far fewer copies are issued, with the
    default policy the cold first step's loads of neighbouring pinned tensors merge; the schedule and every logit are
    unchanged."""
    cfg = replace(si.CONFIGS[1], T=4)
    lay, pool, s, blobs, T = setup(cfg, bits=bits)
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * T, dtype=np.int32).reshape(cfg.B, T) * 311 + 9) % cfg.V
    n_h2d = sum(1 for k in range(0, len(blobs["commands"]), 45) if blobs["commands"][k + 4] == 0)
    out = {}
    for enable in (1, 0):
        tb.k_merge_copies(enable)
        logits, _ = r.generate(prompt, T, forced=forced)
        out[enable] = (logits, s.ctx.copies_issued())
    tb.k_merge_copies(1)
    assert s.ctx.plan_blobs() == blobs
    s.close()
    for a, b in zip(out[1][0], out[0][0]):
        assert np.array_equal(a, b)
    assert out[0][1] == n_h2d                      # switched off: one copy per load command
    # (from the plan alone: 0.62 of the commands with nothing pinned, 0.82 with the default policy - runs of neighbours that
    # need no new wait, mostly in the cold first step)
    assert out[1][1] <= (0.75 if bits == tb.BIT_ZC else 0.95) * n_h2d, (out[1][1], n_h2d)


_CFG2 = {}


def config2_material():
    """Pool (pinned, filled on the GPU, bit-identical to the numpy generator) and oracle weights of config 2, built once."""
    if not _CFG2:
        cfg = si.CONFIGS[2]
        lay = si.build_layout(cfg)
        pool = pinned_pool(lay.pool_bytes)
        si.fill_pool_torch(lay, pool, device="cuda:0")
        u16 = pool.numpy().view(np.uint16)
        W = {}
        for (kind, layer, expert, rows, cols) in si.weight_matrices(cfg):
            parts = [u16[t.pool_off // 2: t.pool_off // 2 + t.rows * t.cols].reshape(t.rows, t.cols) for t in lay.blocks(kind, layer, expert)]
            W[(kind, layer, expert)] = np.concatenate(parts, axis=0) if len(parts) > 1 else parts[0].copy()
        _CFG2.update(cfg=cfg, lay=lay, pool=pool, W=W)
    return _CFG2["cfg"], _CFG2["lay"], _CFG2["pool"], _CFG2["W"]


def test_config_2_prefill_and_first_decode_steps_match_oracle():
    """16 layers deep, the bf16 rounding points decorrelate any two implementations whose summation order differs:
    the oracle itself moves by 5.1e-2 (max) / 1.4e-2 (mean rel) between float32 and float64 accumulation, above the
    stated 3e-2 / 1e-2.  The gate is therefore the larger of the stated tolerance and twice that floor; the
    cascade-free check of the same configuration is the lockstep test."""
    cfg, lay, pool, W = config2_material()
    n_dec = 3
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED)
    s.plan(T=n_dec)
    om = forward.OracleModel(cfg, W, dtype=np.float32)
    prompt = si.prompt_tokens(cfg)
    ref, toks = om.generate(prompt, n_dec)
    r = Runner(s, cfg.B * cfg.S)
    got, _ = r.generate(prompt, n_dec, forced=toks)
    fl_max, fl_rel = precision_floor(2)
    worst_abs = max(float(np.abs(a - b).max()) for a, b in zip(got, ref))
    worst_rel = max(float(np.abs(a - b).mean() / np.abs(b).mean()) for a, b in zip(got, ref))
    print(f"config 2 free-running logits error: max abs {worst_abs:.3e} (oracle float32-vs-float64 floor {fl_max:.3e}, stated {MAX_ABS:.0e}), "
          f"mean relative {worst_rel:.3e} (floor {fl_rel:.3e}, stated {MEAN_REL:.0e})")
    check_logits(got, ref, max(MAX_ABS, 2 * fl_max), max(MEAN_REL, 2 * fl_rel))
    assert all(np.argmax(a[0]) == np.argmax(b[0]) or abs(np.sort(b[0])[-1] - np.sort(b[0])[-2]) < 2 * fl_max for a, b in zip(got, ref))
    s.close()


def test_managed_variants_give_the_same_bits_as_the_explicit_ring():
    """Same kernels reading a cudaMallocManaged pool in place (demand paging, prefetch/advise hints, and the
    object-level prefetcher that asks for whole segments): only the placement mechanism differs, so logits must be
    bitwise equal to the explicit engine's."""
    from paper_2609_06172_b200 import uvm_baseline
    cfg = replace(si.CONFIGS[1], T=4)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 577 + 11) % cfg.V
    lay, pool, s, blobs, T = setup(cfg)
    ref, _ = Runner(s, cfg.B * cfg.S).generate(prompt, T, forced=forced)
    s.close()
    mp = uvm_baseline.ManagedPool(lay.pool_bytes)
    try:
        si.fill_pool(lay, mp.numpy())
        for var in (tb.VAR_MANAGED_DEMAND, tb.VAR_MANAGED_HINTS, tb.VAR_MANAGED_OBJECT):
            sm = Session(lay, MACHINE, pool_base=mp.ptr, pool_flags=tb.POOL_MANAGED)
            sm.plan(T=T, variant=var)
            if var == tb.VAR_MANAGED_OBJECT:
                with pytest.raises(tb.TgpError):
                    sm.ctx.set_object_bytes(4096)                             # below the 64 KiB minimum
                sm.ctx.set_object_bytes(1 << 20)
            r = Runner(sm, cfg.B * cfg.S, arena=False)
            tb.managed_evict(mp.ptr, lay.pool_bytes)
            got, _ = r.generate(prompt, T, forced=forced)
            for a, b in zip(got, ref):
                assert np.array_equal(a, b)
            if var == tb.VAR_MANAGED_OBJECT:
                # the prefetcher asks for whole 1 MiB segments: at least every touched byte, at most the pool per op
                r.reset()
                st = r.step(tb.PREFILL, np.ascontiguousarray(prompt, dtype=np.int32), cfg.S, want_stats=True)
                acc = [a for o in sm.ctx.trace_ops() if o[0] == 0 for a in o[6]]
                whole = sum(t.size for t in lay.tensors if t.kind not in (si.K_EMBED, si.K_KT, si.K_VT))      # read whole by a prefill
                assert st.zc_bytes == 0 and st.d2h_bytes == 0
                assert 0.9 * whole <= st.h2d_bytes <= sum(lay.tensors[a[0]].size + (2 << 20) for a in acc)
                r.sync()
            # KV tiles were written in place: start from zeros again for the next variant
            sm.close()
            si.fill_pool(lay, mp.numpy())
        # a pinned pool cannot run a managed variant: state error, not a fault
        lay2, pool2, s2, _, _ = setup(cfg)
        s2.ctx.set_variant(tb.VAR_MANAGED_DEMAND, 7)
        s2.ctx.model_trace(cfg.S, T)
        s2.ctx.plan()
        r2 = Runner(s2, cfg.B * cfg.S)
        with pytest.raises(tb.TgpError) as ei:
            r2.step(tb.PREFILL, prompt, cfg.S)
        assert ei.value.code == tb.E_STATE
        s2.close()
    finally:
        torch.cuda.synchronize()
        mp.free()


MOE = si.ModelConfig("moe_small", L=2, d=256, Hq=4, Hkv=2, Dh=64, F=512, V=512, B=3, S=9, T=4, TK=4, E=4, topk=2, seed=77,
                     budget_rule="half_w")


def _run_steps(r, cfg, prompt, forced, T):
    """prefill + T teacher-forced decode steps with statistics; returns (logits per step, mismatches per step)."""
    r.reset()
    out, mism = [], []
    st = r.step(tb.PREFILL, np.ascontiguousarray(prompt, dtype=np.int32), cfg.S, want_stats=True)
    for t in range(T + 1):
        out.append(r.logits.cpu().numpy().copy())
        mism.append(st.n_mismatch)
        if t < T:
            st = r.step(tb.DECODE, np.ascontiguousarray(forced[:, t:t + 1], dtype=np.int32), 1, want_stats=True)
    r.sync()
    return out, mism


def test_moe_profile_pass_planned_run_and_mismatch_fallback():
    """Mixture-of-experts path: (1) a profile pass with every expert traced records the routed-token counts, which
    must equal the oracle's routing; (2) the run planned from that profile matches the oracle's logits with no
    fallback; (3) with an expert missing from the trace the engine fetches it synchronously, counts the mismatch,
    and still produces the same logits."""
    cfg = MOE
    lay = si.build_layout(cfg, cap=64 << 10)
    bias = si.router_bias(cfg)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    om = forward.OracleModel(cfg, si.weights_as_bits(lay), bias)
    prompt = si.prompt_tokens(cfg)
    ref, toks = om.generate(prompt, cfg.T)
    want_counts = np.array([[c.tolist() for c in step] for step in om.expert_counts], dtype=np.uint32)     # [steps, L, E]
    assert want_counts.shape == (1 + cfg.T, cfg.L, cfg.E) and (want_counts.sum(axis=2) == cfg.topk * np.array([cfg.B * cfg.S] + [cfg.B] * cfg.T)[:, None]).all()
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED, router_bias=bias)
    # (1) profile pass: all experts traced
    s.plan(expert_counts=np.ones_like(want_counts))
    r = Runner(s, cfg.B * cfg.S)
    got, mism = _run_steps(r, cfg, prompt, toks, cfg.T)
    assert sum(mism) == 0
    counts = s.ctx.expert_counts(cfg.L, cfg.E)
    assert np.array_equal(counts, want_counts)
    check_logits(got, ref)
    # (2) plan from the profile: only the experts in use are staged
    blobs_all = s.ctx.plan_blobs()
    blobs = s.plan(expert_counts=counts)
    ops, steps = trace.run_trace(lay, expert_counts=want_counts)
    want = policy.plan(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget).blobs()
    assert blobs == want
    validate.check(lay.tensors, ops, steps, lay.budget, blobs)
    got2, mism2 = _run_steps(r, cfg, prompt, toks, cfg.T)
    assert sum(mism2) == 0
    check_logits(got2, ref)
    if (want_counts == 0).any():
        assert len(blobs["commands"]) < len(blobs_all["commands"])
    # (3) drop one expert that is in use from the trace of the first decode step, layer 1
    e_used = int(np.argmax(want_counts[1, 1]))
    wrong = counts.copy()
    wrong[1, 1, e_used] = 0
    s.plan(expert_counts=wrong)
    got3, mism3 = _run_steps(r, cfg, prompt, toks, cfg.T)
    assert mism3[1] == 1 and sum(mism3) == 1
    check_logits(got3, ref)
    s.close()


def test_moe_decode_groups_expert_blocks_with_the_same_bits():
    """Expert products are grouped like dense ones (gate and up pieces of one expert, then its down pieces, with the
    gather before and the gate-scaled scatter after): fewer launches, identical logits, no fallback."""
    cfg = MOE
    lay = si.build_layout(cfg, budget=64 << 20, cap=64 << 10)          # everything resident: every group forms
    bias = si.router_bias(cfg)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED, router_bias=bias)
    s.plan(expert_counts=np.ones((1 + cfg.T, cfg.L, cfg.E), dtype=np.uint32))
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 389 + 5) % cfg.V
    runs = {}
    for enable in (1, 0):
        tb.k_gemm_group_select(enable)
        r.reset()
        r.step(tb.PREFILL, prompt, cfg.S)
        logits, launches = [], 0
        for t in range(cfg.T):
            st = r.step(tb.DECODE, np.ascontiguousarray(forced[:, t:t + 1]), 1, want_stats=True)
            assert st.n_mismatch == 0
            launches += st.n_launches
            logits.append(r.logits.cpu().numpy().copy())
        runs[enable] = (logits, launches)
    tb.k_gemm_group_select(1)
    s.close()
    for a, b in zip(runs[1][0], runs[0][0]):
        assert np.array_equal(a, b)
    assert runs[1][1] < runs[0][1]


def _weights_from_pool(lay, pool):
    u16 = pool.numpy().view(np.uint16)
    W = {}
    for (kind, layer, expert, rows, cols) in si.weight_matrices(lay.cfg):
        parts = [u16[t.pool_off // 2: t.pool_off // 2 + t.rows * t.cols].reshape(t.rows, t.cols) for t in lay.blocks(kind, layer, expert)]
        W[(kind, layer, expert)] = np.concatenate(parts, axis=0) if len(parts) > 1 else parts[0].copy()
    return W


def test_llama_8b_widths_at_two_layers_lockstep_parity():
    """Full widths of the 8B shape (d 4096, FFN 14336, vocabulary 128256, head dimension 128, weights split into 32 MiB
    sub-range blocks) at two layers and a short prompt, half the weights resident: prefill of 2 x 136 tokens (tcgen05
    GEMMs and attention with a ragged last query tile) and three decode steps at batch 2.  Checked in lockstep: every
    bf16 rounding point is a legal rounding of the oracle's value computed from the GPU's own inputs, and the logits
    that follow from the GPU's codes meet the stated tolerance (free-running, the 128256 logits of this shape differ by
    up to 4.4e-2 after two layers: the rounding cascade, as on the 16-layer benchmark configuration)."""
    cfg = replace(si.CONFIGS[3], L=2, B=2, S=136, T=3, budget_rule="half_w")
    lay = si.build_layout(cfg)
    assert max(t.size for t in lay.tensors if t.kind in (si.K_WG, si.K_WD, si.K_LM)) <= 32 << 20          # blocks, not whole matrices
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool_torch(lay, pool, device="cuda:0")
    worst, flips = _lockstep(cfg, lay, pool, _weights_from_pool(lay, pool), cfg.T, np.float32)
    assert worst < 5e-3
    assert all(v < 0.02 for k, v in flips.items() if k != "o") and flips["o"] < 0.5
    assert tb.k_attn_status() == 0 and tb.k_gemm_status() == 0


def test_mixtral_widths_at_one_layer_match_oracle_batch_of_eight():
    """Full widths of the Mixtral shape (8 experts of 14336, top-2) at one layer, batch 8, free-running: the expert
    products run at the handful of tokens each expert receives (skinny tensor-core GEMV on blocks of few rows), planned
    from a profile pass.  Routing is an fp32 comparison of router logits whose inputs differ between the two sides by
    bf16 rounding flips, so a token whose second and third logits are within FRAGILE of each other may route either
    way: every difference in the routed-token counts must be explained by such tokens, and the logits of every
    sequence whose deciding (last-position) token is not fragile are compared unconditionally - at one layer a token's
    routing reaches no other position's logits."""
    FRAGILE = 2e-2
    cfg = replace(si.CONFIGS[5], L=1, B=8, S=16, T=2, budget_rule="half_w")
    lay = si.build_layout(cfg)
    bias = si.router_bias(cfg)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool_torch(lay, pool, device="cuda:0")
    om = forward.OracleModel(cfg, _weights_from_pool(lay, pool), bias, dtype=np.float32)
    Wr = om.w[(si.K_ROUTER, 0, -1)].astype(np.float64)
    fragile = []                                                  # per step: bool [B, q]

    def hook(name, layer, pre, out):
        if name == "h2":
            rl = np.sort(out.reshape(-1, cfg.d).astype(np.float64) @ Wr.T + np.asarray(bias[layer], dtype=np.float64), axis=-1)
            fragile.append(((rl[:, -2] - rl[:, -3]) < FRAGILE).reshape(out.shape[0], out.shape[1]))
        return out

    om.hook = hook
    prompt = si.prompt_tokens(cfg)
    ref, toks = om.generate(prompt, cfg.T)
    om.hook = None
    want_counts = np.array([[c.tolist() for c in step] for step in om.expert_counts], dtype=np.uint32)
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED, router_bias=bias)
    s.plan(expert_counts=np.ones_like(want_counts))
    r = Runner(s, cfg.B * cfg.S)
    got, mism = _run_steps(r, cfg, prompt, toks, cfg.T)
    counts = s.ctx.expert_counts(cfg.L, cfg.E)
    for k in range(1 + cfg.T):
        moved = int(np.abs(counts[k].astype(np.int64) - want_counts[k].astype(np.int64)).sum())
        assert moved <= 2 * int(fragile[k].sum()), (k, moved, int(fragile[k].sum()))
    s.plan(expert_counts=counts)
    got2, mism2 = _run_steps(r, cfg, prompt, toks, cfg.T)
    assert sum(mism2) == 0
    for a, b in zip(got, got2):
        assert np.array_equal(a, b)                                           # profile pass and planned run: same bits
    compared = 0
    for k in range(1 + cfg.T):
        keep = ~fragile[k][:, -1]                                             # sequences whose last position routes robustly
        compared += int(keep.sum())
        check_logits([got2[k][keep]], [ref[k][keep]])
    assert compared >= (1 + cfg.T) * cfg.B * 3 // 4, compared
    s.close()


def test_mixtral_widths_at_three_layers_lockstep_parity():
    """Full widths of the Mixtral shape at three layers, batch 4, prefill of 4 x 24 tokens and two decode steps, half
    the weights resident, in lockstep: routing counts equal to the oracle's at every step and layer, every rounding
    point a legal rounding, logits within the stated tolerance."""
    cfg = replace(si.CONFIGS[5], L=3, B=4, S=24, T=2, budget_rule="half_w")
    lay = si.build_layout(cfg)
    bias = si.router_bias(cfg)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool_torch(lay, pool, device="cuda:0")
    worst, flips = _lockstep(cfg, lay, pool, _weights_from_pool(lay, pool), cfg.T, np.float32, bias=bias)
    assert worst < 5e-3
    assert all(v < 0.02 for k, v in flips.items() if k != "o") and flips["o"] < 0.5
    assert tb.k_attn_status() == 0 and tb.k_gemm_status() == 0


def test_llama_70b_widths_at_two_layers_lockstep_parity():
    """Full widths of the 70B shape (d 8192, 64 query / 8 KV heads, FFN 28672, vocabulary 128256) at two layers: prefill
    of 2 x 136 tokens and two decode steps at batch 2, half the weights resident, in lockstep."""
    cfg = replace(si.CONFIGS[4], L=2, B=2, S=136, T=2, budget_rule="half_w")
    lay = si.build_layout(cfg)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool_torch(lay, pool, device="cuda:0")
    worst, flips = _lockstep(cfg, lay, pool, _weights_from_pool(lay, pool), cfg.T, np.float32)
    assert worst < 5e-3
    assert all(v < 0.02 for k, v in flips.items() if k != "o") and flips["o"] < 0.5
    assert tb.k_attn_status() == 0 and tb.k_gemm_status() == 0


def test_llama_8b_full_depth_lockstep_parity_reduced_tokens():
    """The 8B configuration at its full depth (all 32 layers), full widths and its 8 GiB budget (2x oversubscribed), with
    reduced tokens - one sequence, prompt of 16, four decode steps - because a full-size CPU forward pass would take
    hours.  Lockstep: every rounding point of all 32 layers element by element, logits within the stated tolerance."""
    cfg = replace(si.CONFIGS[3], B=1, S=16, T=4)
    lay = si.build_layout(cfg)
    assert lay.budget == 8 << 30 and cfg.L == 32 and lay.pool_bytes > 1.8 * lay.budget          # weights alone: 1.87x the budget
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool_torch(lay, pool, device="cuda:0")
    worst, flips = _lockstep(cfg, lay, pool, _weights_from_pool(lay, pool), cfg.T, np.float32)
    assert worst < 5e-3
    assert all(v < 0.02 for k, v in flips.items() if k != "o") and flips["o"] < 0.5
    assert tb.k_attn_status() == 0 and tb.k_gemm_status() == 0


def test_layer_aliased_host_pool_runs_like_a_pool_with_repeated_layers():
    """The host pool for shapes too large to page-lock (layers l and l + 2 on the same physical pages, page-locked mapping
    by mapping) against an ordinary pinned pool that holds the same bytes: same plan, bitwise equal logits."""
    from paper_2609_06172_b200.runner import AliasedPool
    cfg = replace(si.CONFIGS[1], L=4, d=1024, F=4096, Hq=16, Hkv=16, T=3, budget_rule="half_w")
    lay = si.build_layout(cfg)
    ap = AliasedPool(lay, 2)
    ap.page_lock()
    try:
        si.fill_pool(lay, ap.numpy())                        # layers 2, 3 are written last: layers 0, 1 now hold their values too
        pool = pinned_pool(lay.pool_bytes)
        pool.numpy()[:] = ap.numpy()
        prompt = si.prompt_tokens(cfg)
        forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 131 + 7) % cfg.V
        outs = []
        for base in (pool.data_ptr(), ap.data_ptr()):
            s = Session(lay, MACHINE, pool_base=base, pool_flags=tb.POOL_PINNED)
            blobs = s.plan(T=cfg.T)
            got, _ = Runner(s, cfg.B * cfg.S).generate(prompt, cfg.T, forced=forced)
            outs.append((blobs, got))
            s.close()
        assert outs[0][0] == outs[1][0]
        for a, b in zip(outs[0][1], outs[1][1]):
            assert np.array_equal(a, b) and np.isfinite(a).all()
        w = {t.layer: t for t in lay.tensors if t.kind == si.K_WQ}
        assert np.array_equal(ap.numpy()[w[0].pool_off: w[0].pool_off + 64], ap.numpy()[w[2].pool_off: w[2].pool_off + 64])
    finally:
        torch.cuda.synchronize()
        ap.close()


def test_router_topk_ties_and_single_expert_equals_dense():
    """E = 1, top-1 routes every token to the one expert with gate 1: same logits as the dense model with those weights."""
    dense = replace(MOE, E=0, topk=0, L=1)
    moe1 = replace(MOE, E=1, topk=1, L=1)
    lay_d, lay_m = si.build_layout(dense, cap=64 << 10), si.build_layout(moe1, cap=64 << 10)
    pd, pm = pinned_pool(lay_d.pool_bytes), pinned_pool(lay_m.pool_bytes)
    si.fill_pool(lay_d, pd.numpy())
    si.fill_pool(lay_m, pm.numpy())
    # give the single expert the dense FFN's weights (block by block) and share all other weights
    for t in lay_m.tensors:
        key = (t.kind, t.layer, -1 if t.expert == 0 else t.expert)
        if t.kind == si.K_ROUTER or t.kind >= si.K_KT:
            continue
        src = lay_d.blocks(*key)[t.block]
        assert src.size == t.size
        pm.numpy()[t.pool_off:t.pool_off + t.size] = pd.numpy()[src.pool_off:src.pool_off + src.size]
    prompt = si.prompt_tokens(dense)
    forced = (np.arange(dense.B * dense.T, dtype=np.int32).reshape(dense.B, dense.T) * 131 + 5) % dense.V
    sd = Session(lay_d, MACHINE, pool_base=pd.data_ptr(), pool_flags=tb.POOL_PINNED)
    sd.plan()
    a, _ = Runner(sd, dense.B * dense.S).generate(prompt, dense.T, forced=forced)
    sm = Session(lay_m, MACHINE, pool_base=pm.data_ptr(), pool_flags=tb.POOL_PINNED, router_bias=np.zeros((1, 1), np.float32))
    counts = np.array([[[dense.B * dense.S]]] + [[[dense.B]]] * dense.T, dtype=np.uint32)
    sm.plan(expert_counts=counts)
    b, _ = Runner(sm, dense.B * dense.S).generate(prompt, dense.T, forced=forced)
    for x, y in zip(a, b):
        assert np.abs(x - y).max() < 1e-5
    sd.close(), sm.close()


# ---- lockstep parity: every rounding point, no cascade ------------------------------------------------------------
def _bf16_ulp(x):
    ax = np.maximum(np.abs(x.astype(np.float64)), 2.0 ** -120)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


ROUTER_MARGIN = 1e-4      # a token whose second and third router logits are closer than this could route either way


def _lockstep(cfg, lay, pool, W, n_dec, dtype, bias=None):
    """Runs GPU and oracle step by step.  At every bf16 rounding point the oracle is handed the GPU's tensor, checks
    that each element is a legal rounding of the oracle's own pre-rounding value (|gpu - pre| <= ulp/2 plus the
    summation-order slack of that op) and continues from the GPU's codes, so a flipped rounding cannot cascade.
    Mixture of experts (bias given): both routers then see the same bf16 inputs, so the routed-token counts of every
    step and layer must be equal - after checking, as a fact about the seeded inputs, that no token's second and third
    router logits are within ROUTER_MARGIN of each other (fp32 summation order moves a logit by ~1e-6).
    Returns worst logit error and the fraction of roundings that differ from the oracle's, per kind."""
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED, router_bias=bias)
    if cfg.E:
        s.plan(T=n_dec, expert_counts=np.ones((1 + n_dec, cfg.L, cfg.E), dtype=np.uint32))     # every expert traced: nothing falls back
    else:
        s.plan(T=n_dec)
    ops = s.ctx.trace_ops()
    r = Runner(s, cfg.B * cfg.S)
    qd, F, d = cfg.Hq * cfg.Dh, cfg.F, cfg.d
    per_layer = cfg.B * cfg.S * (2 * d + 2 * qd + F * max(1, cfg.topk)) * 2 + 2 * cfg.n_tiles * cfg.B * cfg.Hkv * cfg.TK * cfg.Dh * 2 + (16 + cfg.E) * 256
    tap = torch.empty(per_layer * cfg.L + (1 << 20), dtype=torch.uint8, device="cuda:0")
    om = forward.OracleModel(cfg, W, bias, dtype=dtype)
    W = None                                               # the oracle holds its own converted copy
    Wr = {l: om.w[(si.K_ROUTER, l, -1)].astype(np.float64) for l in range(cfg.L)} if cfg.E else {}
    margins = []
    # slack per rounding point, relative to |pre| + mean|pre|: fp32 summation order and libm vs device exp.  The normed
    # states sit behind the residual stream, which sums tensor-core products of K up to 8192 per layer (their fp32
    # accumulation is not round-to-nearest: ~5e-5 typical, 3e-4 covers the tail of 1e6 elements); the attention output
    # also carries the tensor-core kernel's bf16 rounding of the softmax weights (not mirrored by the oracle)
    # (the tensor cores' fp32 accumulation is not round-to-nearest: its error has a part linear in K, so the points fed
    # directly by a product over K = d get a slack that grows with d beyond 4096)
    kd = 1e-4 * max(1.0, cfg.d / 4096)
    rtol = {"h": 3e-4, "h2": 3e-4, "hf": 3e-4, "q": kd, "k": kd, "v": kd, "a": kd, "o": 4e-3}
    flips = {k: [0, 0] for k in rtol}
    prompt = si.prompt_tokens(cfg)
    worst = 0.0
    r.reset()
    pos0 = 0
    tok = prompt
    for step in range(1 + n_dec):
        q = tok.shape[1]
        s.ctx.set_tap(tap, tap.numel())
        r.step(tb.PREFILL if step == 0 else tb.DECODE, np.ascontiguousarray(tok, dtype=np.int32), q)
        r.sync()
        idx = s.ctx.tap_index()
        host = tap.cpu().numpy()
        got = {}
        seen_h = {}
        for (op, tag, sub, off, nbytes) in idx.tolist():
            layer = ops[op][2]
            a = si.bf16_bits_to_f32(host[off:off + nbytes].view(np.uint16))
            if tag == tb.TAP_H:
                name = "h2" if seen_h.get(layer) else "h"
                seen_h[layer] = True
                got[(name, layer)] = a.reshape(cfg.B, q, d)
            elif tag == tb.TAP_HF:
                got[("hf", -1)] = a.reshape(cfg.B, 1, d)
            elif tag == tb.TAP_Q:
                got[("q", layer)] = a.reshape(cfg.B, q, cfg.Hq, cfg.Dh)
            elif tag in (tb.TAP_KTILE, tb.TAP_VTILE):
                got.setdefault(("k" if tag == tb.TAP_KTILE else "v", layer), {})[sub] = a.reshape(cfg.B, cfg.Hkv, cfg.TK, cfg.Dh)
            elif tag == tb.TAP_O:
                got[("o", layer)] = a.reshape(cfg.B, q, cfg.Hq, cfg.Dh)
            elif tag == tb.TAP_A:
                if cfg.E:
                    got[("a.e%d" % sub, layer)] = a.reshape(-1, F)             # rows routed to expert `sub`, ascending token order
                else:
                    got[("a", layer)] = a.reshape(cfg.B, q, F)

        def hook(name, layer, pre, out, pos0=pos0, q=q):
            if (name, layer) not in got:
                raise AssertionError(("the GPU recorded no activation for this rounding point (routing differs?)", name, layer))
            g = got[(name, layer)]
            if name in ("k", "v"):                         # gather the new positions out of the tapped tiles
                new = np.empty((cfg.B, q, cfg.Hkv, cfg.Dh), dtype=np.float32)
                for p in range(pos0, pos0 + q):
                    new[:, p - pos0] = g[p // cfg.TK][:, :, p % cfg.TK, :]
                g = new
            g = g.reshape(pre.shape)
            name = name.split(".")[0]                      # "a.e3" (expert 3's SwiGLU output) is checked like "a"
            # (the attention output averages rows of V, so its P-rounding error scales with |V| ~ max|o|, not with |o|)
            scale = np.abs(pre).max() if name == "o" else np.abs(pre).mean()
            bound = 0.5 * _bf16_ulp(pre) * (1 + 1e-6) + rtol[name] * (np.abs(pre) + scale)
            bad = np.abs(g.astype(np.float64) - pre.astype(np.float64)) > bound
            assert not bad.any(), (name, layer, int(bad.sum()), float(np.abs(g - pre)[bad].max()))
            flips[name][0] += int((g != out).sum())
            flips[name][1] += g.size
            if name == "h2" and cfg.E:                     # the router's input: how far is every token from a routing tie?
                rl = np.sort(g.reshape(-1, cfg.d).astype(np.float64) @ Wr[layer].T + np.asarray(bias[layer], dtype=np.float64), axis=-1)
                margins.append(float((rl[:, -cfg.topk] - rl[:, -cfg.topk - 1]).min()))
            return g

        om.hook = hook
        ref = om.step(tok, pos0)
        om.hook = None
        if cfg.E:
            assert min(margins) > ROUTER_MARGIN, ("seeded inputs put a token on a routing near-tie: pick another seed", min(margins))
            want_counts = np.array([c.tolist() for c in om.expert_counts[-1]], dtype=np.uint32)
            assert np.array_equal(s.ctx.expert_counts(cfg.L, cfg.E)[step], want_counts), step
        dev = r.logits.cpu().numpy()
        err = np.abs(dev - ref)
        assert err.max() < MAX_ABS and err.mean() / np.abs(ref).mean() < MEAN_REL, (step, err.max())
        worst = max(worst, float(err.max()))
        pos0 += q
        tok = np.argmax(ref, axis=-1).astype(np.int32)[:, None]
    s.ctx.set_tap(None, 0)
    s.close()
    return worst, {k: (v[0] / max(1, v[1])) for k, v in flips.items()}


def test_lockstep_parity_config_1_all_steps():
    cfg = si.CONFIGS[1]
    lay = si.build_layout(cfg)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    worst, flips = _lockstep(cfg, lay, pool, si.weights_as_bits(lay), cfg.T, np.float64)
    assert worst < 1e-3                                    # with the cascade removed the logits agree far inside the stated 3e-2
    assert all(v < 0.02 for k, v in flips.items() if k != "o") and flips["o"] < 0.5


def test_lockstep_parity_config_2_full_size_prefill_and_decode():
    """The benchmark's configuration at full size and in its launch configuration (50 % budget, ring + pins):
    every rounding point of every layer is checked element by element, and the logits meet the stated tolerance."""
    cfg, lay, pool, W = config2_material()
    worst, flips = _lockstep(cfg, lay, pool, W, 2, np.float32)
    assert worst < 5e-3
    assert all(v < 0.02 for k, v in flips.items() if k != "o") and flips["o"] < 0.5


def test_runtime_monitor_replan_from_measured_kernel_times():
    """Second half of the paper's runtime monitor: kernel timestamps of a real run re-classify the ops, the schedule is
    rebuilt, and (the log being integers) the oracle's planner rebuilds the identical schedule from the same log.
    Placement changes, results do not: logits are bitwise equal before and after the re-plan."""
    cfg = si.CONFIGS[1]
    lay, pool, s, blobs, T = setup(cfg)
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * T, dtype=np.int32).reshape(cfg.B, T) * 313 + 7) % cfg.V
    before, _ = r.generate(prompt, T, forced=forced)
    ops, steps = trace.run_trace(lay)
    ns = np.zeros(len(ops), dtype=np.uint64)
    r.reset()
    s.ctx.set_op_timing(True)
    for k in range(1 + T):
        tok = prompt if k == 0 else np.ascontiguousarray(forced[:, k - 1:k], dtype=np.int32)
        r.step(tb.PREFILL if k == 0 else tb.DECODE, tok, tok.shape[1], want_stats=True)
        first, ms = s.ctx.op_times()
        ns[first:first + len(ms)] = np.maximum(1, np.round(ms.astype(np.float64) * 1e6)).astype(np.uint64)
    s.ctx.set_op_timing(False)
    r.sync()
    assert (ns > 0).all()
    s.ctx.set_measured_times(ns)
    s.ctx.plan()
    got = s.ctx.plan_blobs()
    want = policy.plan(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget, measured_ns=ns.tolist()).blobs()
    assert got == want
    validate.check(lay.tensors, ops, steps, lay.budget, got)
    # microsecond kernels on a 55 GB/s link: small tensors' ops stop being link-bound
    assert got["classes"] != blobs["classes"]
    after, _ = r.generate(prompt, T, forced=forced)
    for a, b in zip(before, after):
        assert np.array_equal(a, b)
    s.close()


def test_replan_that_keeps_the_pins_switches_twice_without_reloading_them():
    """tgp_set_replan_keep: at a switch the pinned tensors that are on the device stay where they are.  Two switches in one
    run (the second from a plan that itself kept pins): each tail schedule is bit for bit the oracle's for the resident set
    read off the plan in use, passes the validator started with that set resident, and places none of the kept tensors;
    the step after a switch copies far fewer bytes than the same step after a cold switch; the logits of every step -
    KV tiles written before a switch are read after it from where they stayed - equal those of the run that never
    switched, bit for bit."""
    cfg = si.CONFIGS[1]
    lay, pool, s, blobs, T = setup(cfg)
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * T, dtype=np.int32).reshape(cfg.B, T) * 211 + 5) % cfg.V
    plain, _ = r.generate(prompt, T, forced=forced)
    ops, steps = trace.run_trace(lay)
    mach = policy.Machine(**MACHINE)
    nt = len(lay.tensors)

    def resident_of(b, first_op):
        P = validate.parse(b, nt)
        placed = {}
        for (seq, kind, t, nb, po, ao, w, f, rel) in P["cmds"]:
            if kind != validate.CMD_D2H:
                placed.setdefault((t, ao), f)
        return {t: o for t, o in P["pins"] if placed.get((t, o), -1) < first_op}

    def run(keep, boundaries):
        r.reset()
        s.ctx.set_replan_keep(keep)
        out, h2d, tails = [], [], {}
        for k in range(1 + T):
            if k + 2 in boundaries:
                s.ctx.replan_begin(k + 2)
            if k in boundaries:
                in_use = s.ctx.plan_blobs()
                s.ctx.replan_commit()
                tails[k] = (in_use, s.ctx.plan_blobs())
            tok = prompt if k == 0 else np.ascontiguousarray(forced[:, k - 1:k], dtype=np.int32)
            st = r.step(tb.PREFILL if k == 0 else tb.DECODE, tok, tok.shape[1], want_stats=True)
            h2d.append(st.h2d_bytes)
            out.append(r.logits.cpu().numpy().copy())
        r.sync()
        return out, h2d, tails

    cold_out, cold_h2d, _ = run(False, (4, 9))
    keep_out, keep_h2d, tails = run(True, (4, 9))
    for k, (in_use, tail) in tails.items():
        res = resident_of(in_use, steps[k][1])
        assert tail == policy.plan_tail(lay.tensors, ops, steps, mach, lay.budget, k, resident=res).blobs()
        validate.check(lay.tensors, ops, steps, lay.budget, tail, first_step=k, resident=res)
        P = validate.parse(tail, nt)
        kept = {t for t, o in res.items() if dict(P["pins"]).get(t) == o}
        assert kept and not ({c[2] for c in P["cmds"] if c[1] != validate.CMD_D2H} & kept)
        assert keep_h2d[k] < 0.6 * cold_h2d[k]                      # the cold switch reloads the pinned half of the pool in this step
    for a, b, c in zip(keep_out, cold_out, plain):
        assert np.array_equal(a, c) and np.array_equal(b, c)
    s.ctx.set_replan_keep(False)
    again, _ = r.generate(prompt, T, forced=forced)
    assert s.ctx.plan_blobs() == blobs
    for a, b in zip(again, plain):
        assert np.array_equal(a, b)
    s.close()


@pytest.mark.parametrize("budget", [None, 3 << 20])
def test_replan_in_the_middle_of_a_run_switches_plans_at_a_step_boundary(budget):
    """Runtime monitor while the run is under way: after decode step 3 the timing log so far is handed to the planner,
    which plans steps 6.. on a helper thread while steps 4 and 5 still execute from the old plan; at the boundary the
    engine drains, writes the written pinned KV tiles back and switches.  The tail schedule is bit for bit what the
    oracle's tail planner gives for the same integer log and passes the validator; logits of every step equal those
    of the un-switched run bit for bit; a reset brings the whole-run plan back."""
    cfg = si.CONFIGS[1]
    lay, pool, s, blobs, T = setup(cfg, budget=budget)
    r = Runner(s, cfg.B * cfg.S)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * T, dtype=np.int32).reshape(cfg.B, T) * 211 + 5) % cfg.V
    plain, _ = r.generate(prompt, T, forced=forced)
    ops, steps = trace.run_trace(lay)
    boundary, measured_through = 6, 3
    ns = np.zeros(len(ops), dtype=np.uint64)
    got = []
    r.reset()
    s.ctx.set_op_timing(True)
    for k in range(1 + T):
        if k == measured_through + 1:
            # the log so far; ops still to come take the time of the same op in the last measured decode step
            s.ctx.set_op_timing(False)
            o0, n = steps[measured_through][1], steps[measured_through][2]
            for j in range(measured_through + 1, len(steps)):
                assert steps[j][2] == n
                ns[steps[j][1]: steps[j][1] + n] = ns[o0: o0 + n]
            s.ctx.replan_begin(boundary, ns)                            # plans on a helper thread from here on
        if k == boundary:
            s.ctx.replan_commit()
            tail = s.ctx.plan_blobs()
        tok = prompt if k == 0 else np.ascontiguousarray(forced[:, k - 1:k], dtype=np.int32)
        r.step(tb.PREFILL if k == 0 else tb.DECODE, tok, tok.shape[1], want_stats=True)
        if k <= measured_through:
            first, ms = s.ctx.op_times()
            ns[first:first + len(ms)] = np.maximum(1, np.round(ms.astype(np.float64) * 1e6)).astype(np.uint64)
        got.append(r.logits.cpu().numpy().copy())
    r.sync()
    want = policy.plan_tail(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget, boundary, measured_ns=ns.tolist()).blobs()
    assert tail == want
    validate.check(lay.tensors, ops, steps, lay.budget, tail, first_step=boundary)
    assert tail["commands"] != blobs["commands"]
    for a, b in zip(got, plain):
        assert np.array_equal(a, b)
    # the KV tiles the old plan had pinned were written back at the switch: the pool holds their data
    old_pins = {t for t, _ in np.frombuffer(blobs["pins"][:-16], dtype=np.dtype([("t", "<u4"), ("o", "<u8")])).tolist()}
    written = {t for o in ops[:steps[boundary][1]] for (t, m, _) in o.acc if m & 2}
    host = pool.numpy()
    assert old_pins & written
    assert all(host[lay.tensors[t].pool_off: lay.tensors[t].pool_off + lay.tensors[t].size].any() for t in old_pins & written)
    # after a reset the whole-run plan is in use again
    again, _ = r.generate(prompt, T, forced=forced)
    assert s.ctx.plan_blobs() == blobs
    for a, b in zip(again, plain):
        assert np.array_equal(a, b)
    s.close()


def test_windowed_pin_reservation_runs_bitwise_equal_to_a_resident_run():
    """Slots of KV tiles that are born in later decode steps house weight blocks until then (tenants are loaded once,
    used in place, and give the slot up before the tile's first write): the plan differs from the static one, moves
    fewer bytes, equals the oracle's bit for bit, and the logits of all 41 steps equal those of a run with everything
    resident."""
    cfg = replace(si.CONFIGS[1], B=4, S=30, T=40, TK=16)
    prompt = si.prompt_tokens(cfg)
    forced = (np.arange(cfg.B * cfg.T, dtype=np.int32).reshape(cfg.B, cfg.T) * 733 + 1) % cfg.V
    outs, moved = {}, {}
    for name, budget, bits in (("windowed", None, 15), ("static", None, 7), ("resident", 64 << 20, 15)):
        lay, pool, s, blobs, T = setup(cfg, budget=budget, bits=bits, cap=16 << 10)
        ops, steps = trace.run_trace(lay)
        assert blobs == policy.plan(lay.tensors, ops, steps, policy.Machine(**MACHINE), lay.budget, bits=bits).blobs()
        validate.check(lay.tensors, ops, steps, lay.budget, blobs)
        moved[name] = int(np.frombuffer(blobs["totals"], dtype="<u8").reshape(-1, 4)[:, 0].sum())
        outs[name], _ = Runner(s, cfg.B * cfg.S).generate(prompt, T, forced=forced)
        s.close()
    assert moved["windowed"] < moved["static"]
    for a, b, c in zip(outs["windowed"], outs["static"], outs["resident"]):
        assert np.array_equal(a, c) and np.array_equal(b, c)


def test_whole_run_cuda_graph_replays_bit_identically():
    """The planned run (copies, kernels, cross-stream ordering, device-side argmax feedback) captured as one CUDA graph:
    two replays give exactly the logits and tokens of the plain stepped run, and call-order mistakes are state errors."""
    cfg = replace(si.CONFIGS[1], B=2, S=21, T=9, TK=8)
    lay, pool, s, blobs, T = setup(cfg, cap=128 << 10)
    r = Runner(s, cfg.B * cfg.S)
    prompt = torch.from_numpy(si.prompt_tokens(cfg)).pin_memory()
    plain, toks = r.generate(prompt.numpy(), T)                      # free-running greedy decode, stepped
    with pytest.raises(tb.TgpError) as ei:
        s.ctx.run_graph_launch(r.compute)                            # nothing captured yet
    assert ei.value.code == tb.E_STATE
    r.capture_run(prompt, T)
    with pytest.raises(tb.TgpError):
        s.ctx.run_capture_end()                                      # not capturing any more
    for _ in range(2):
        r.logits.zero_()
        r.argmax.zero_()
        r.replay()
        r.sync()
        assert np.array_equal(r.logits.cpu().numpy(), plain[-1])
        assert np.array_equal(r.argmax.cpu().numpy(), np.argmax(plain[-1], axis=-1).astype(np.int32))
    # back to plain stepping after a reset
    again, toks2 = r.generate(prompt.numpy(), T)
    assert np.array_equal(again[-1], plain[-1]) and np.array_equal(toks, toks2)
    s.close()


def test_whole_run_cuda_graph_with_cluster_launched_and_tma_kernels():
    """Graph capture of a run whose prefill is large enough for the cluster-launched paired GEMM and the TMA-fed tcgen05
    attention (tensor maps are kernel arguments baked into the graph): the replay equals the stepped run bit for bit."""
    cfg = replace(si.CONFIGS[1], L=2, d=1024, F=4096, Hq=16, Hkv=4, V=8192, B=4, S=512, T=2, TK=128, budget_rule="half_w")
    lay, pool, s, blobs, T = setup(cfg)
    r = Runner(s, cfg.B * cfg.S)
    prompt = torch.from_numpy(si.prompt_tokens(cfg)).pin_memory()
    plain, toks = r.generate(prompt.numpy(), T)
    r.capture_run(prompt, T)
    for _ in range(2):
        r.logits.zero_()
        r.replay()
        r.sync()
        assert np.array_equal(r.logits.cpu().numpy(), plain[-1])
    assert tb.k_gemm_status() == 0 and tb.k_attn_status() == 0
    s.close()


def test_edge_shapes_single_token_prompt_no_decode_and_maximum_tile_count():
    """Degenerate sizes: a prompt of one token with no decode step, and a context that needs all 64 KV tiles a kernel
    can address (TK = 1), both against the oracle; requests beyond the workspace or max_len are refused."""
    one = si.ModelConfig("one", L=2, d=128, Hq=2, Hkv=2, Dh=64, F=256, V=300, B=1, S=1, T=0, TK=4, seed=9, budget_rule="half_w_kv")
    lay = si.build_layout(one, cap=16 << 10)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED)
    s.plan()
    ref, _ = forward.OracleModel(one, si.weights_as_bits(lay)).generate(si.prompt_tokens(one), 0)
    r = Runner(s, 1)
    got, toks = r.generate(si.prompt_tokens(one), 0)
    assert len(got) == 1 and toks.shape == (1, 0)
    check_logits(got, ref)
    with pytest.raises(tb.TgpError) as ei:
        r.step(tb.DECODE, None, 1)                                   # the plan has no decode step
    assert ei.value.code == tb.E_STATE
    s.close()
    many = si.ModelConfig("tiles", L=1, d=128, Hq=4, Hkv=2, Dh=64, F=256, V=300, B=2, S=40, T=24, TK=1, seed=10, budget_rule="half_w_kv")
    assert many.n_tiles == 64
    lay = si.build_layout(many, cap=16 << 10)
    pool = pinned_pool(lay.pool_bytes)
    si.fill_pool(lay, pool.numpy())
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED)
    s.plan()
    om = forward.OracleModel(many, si.weights_as_bits(lay))
    prompt = si.prompt_tokens(many)
    ref, toks = om.generate(prompt, many.T)
    r = Runner(s, many.B * many.S)
    got, _ = r.generate(prompt, many.T, forced=toks)
    check_logits(got, ref)
    r.reset()
    with pytest.raises(tb.TgpError) as ei:
        r.step(tb.PREFILL, np.zeros((many.B, many.S + 1), np.int32), many.S + 1)      # more tokens than the workspace holds
    assert ei.value.code == tb.E_INVAL
    s.close()
