#!/usr/bin/env python
"""Benchmark of the hot path: tokens/s at a fixed device budget.

One "step" is one whole pass of the path over one batch: prefill of the prompt, then every decode step,
from a cold arena, with the weight/KV pool in pinned host memory and a device budget of half the weights
(the Llama-1B-shaped configuration, 2x oversubscribed).  `value` is tokens/s with the device feeding its own
argmax back (no host round trip per token); `e2e` puts the host in the loop: tokens come from pinned host
memory every step and each step's argmax (and the final logits) are read back.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config 2]

With N > 1 (torchrun) every rank runs an independent replica on its own GPU (the path does not shard:
no collective on the data path); the line reports the whole-job rate over the slowest rank.
`--impl reference` times the CPU oracle on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
from dataclasses import replace
import json
import os
import struct
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
import seeded_inputs as si  # noqa: E402

# roofline constants frozen for the planner (integers): sustained bf16 peak and HBM copy bandwidth measured on
# this machine's B200, pinned host-link bandwidth at 256 MiB measured by this build (profiles/host_link.md)
MACHINE = dict(peak_flops=1362800000000000, hbm_Bps=6541100000000, h2d_Bps=55570000000, d2h_Bps=56900000000)
OP_NAMES = ["embed", "rmsnorm", "gemm", "rope_kv", "attn", "swiglu", "router", "argmax"]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=j["hbm_gbs"], bf16_tflops=j["bf16_tflops"], bf16_sustained=j.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) >= 7:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_weights_from_pool(lay, pool_u8):
    """bf16 bit matrices per logical weight, re-joined from the pool's blocks (input data for the oracle)."""
    u16 = pool_u8.view(np.uint16)
    out = {}
    for (kind, layer, expert, rows, cols) in si.weight_matrices(lay.cfg):
        parts = [u16[t.pool_off // 2: t.pool_off // 2 + t.rows * t.cols].reshape(t.rows, t.cols) for t in lay.blocks(kind, layer, expert)]
        out[(kind, layer, expert)] = np.concatenate(parts, axis=0) if len(parts) > 1 else parts[0]
    return out


def make_oracle(lay, weights):
    from oracle.forward import OracleModel
    cfg = lay.cfg
    return OracleModel(cfg, weights, si.router_bias(cfg) if cfg.E else None, dtype=np.float32)


def time_oracle(lay, om, sample_S, sample_T):
    """Oracle (float32 accumulate, numpy) on a bounded sample: prefill of sample_S prompt tokens + sample_T decode steps.
    The model (weights already converted) is built by the caller, outside the timed region."""
    cfg = lay.cfg
    prompt = si.prompt_tokens(cfg)[:, :sample_S]
    t0 = time.perf_counter()
    om.generate(prompt, sample_T)
    dt = time.perf_counter() - t0
    return cfg.B * (sample_S + sample_T) / dt, dt


def gemm_shapes_of_step(lay, M, pinned=None):
    """(n, K, residual, M) of every weight-block launch of one step, in trace order (lm_head at M = B).  Consecutive dense
    blocks that read the same activations and carry the same non-zero tgp_k_gemm_group_key() share a launch, as in
    tgp_step(); n is then the tuple of their row counts.  pinned: ids of the tensors the plan keeps resident - a block
    that is staged through the ring ends its launch, as in tgp_step() (a later copy waits for its slot); None: every
    block resident."""
    from paper_2609_06172_b200 import binding as tb
    cfg = lay.cfg
    out = []

    def emit(blocks, res, m):
        """blocks: weight blocks in op order, all multiplied with the same activations (new ones: another kernel wrote them
        just before the first of these launches)."""
        run = []
        first = len(out)
        def flush():
            if len(run) == 1:
                out.append((run[0].rows, run[0].cols, res, m))
            elif run:
                out.append((tuple(t.rows for t in run), run[0].cols, res, m))
            run.clear()
        for t in blocks:
            key = tb.k_gemm_group_key(m, t.rows, t.cols) if m <= 32 else 0
            if run and (not key or key != run_key[0] or t.cols != run[0].cols or len(run) == GROUP_MAX):
                flush()
            if not key:
                out.append((t.rows, t.cols, res, m))
                continue
            if not run:
                run_key[0] = key
            run.append(t)
            if pinned is not None and t.tid not in pinned:
                flush()
        flush()
        if len(out) > first:
            new_acts.add(first)

    run_key = [0]
    new_acts = set()          # indices of the launches that are the first over their activations
    gemm_shapes_of_step.new_acts = new_acts
    for l in range(cfg.L):
        emit([t for kind in (si.K_WQ, si.K_WK, si.K_WV) for t in lay.blocks(kind, l)], 0, M)
        emit(lay.blocks(si.K_WO, l), 1, M)
        if cfg.E:                                             # MoE: tokens spread evenly over the experts (top-k picks each)
            me = max(1, M * cfg.topk // cfg.E)
            for e in range(cfg.E):
                emit([t for kind in (si.K_WG, si.K_WU) for t in lay.blocks(kind, l, e)], 0, me)
                emit(lay.blocks(si.K_WD, l, e), 0, me)
        else:
            emit([t for kind in (si.K_WG, si.K_WU) for t in lay.blocks(kind, l)], 0, M)
            emit(lay.blocks(si.K_WD, l), 1, M)
    emit(lay.blocks(si.K_LM), 0, cfg.B)
    return out


GROUP_MAX = 8     # TGP_GEMM_GROUP_MAX


def kernel_loop(lay, M, reps, device, cold_bytes=1 << 30, min_seconds=1.5, pinned=None):
    """Times the weight-block products of one step back to back on one stream, every launch reading a different
    (cold) region of a buffer larger than L2, exactly as tgp_step launches them (same entry point, shapes, M).
    The whole-step loop is replayed for at least min_seconds (and at least `reps` replays when min_seconds is 0: the small
    form for ncu captures).  Returns (avg seconds per launch, algorithmic bytes per launch, flops per launch, launches
    per rep, per-shape table with the name of the kernel the library launched for each shape)."""
    import torch
    from paper_2609_06172_b200 import binding as tb
    cfg = lay.cfg
    shapes = gemm_shapes_of_step(lay, M, pinned)
    # random operands with the weights' distribution: constant data would toggle few wires, draw little power and let
    # a seconds-long tensor-core loop run at clocks the real step (random weights, power-capped) never sees
    gen = torch.Generator(device=device)
    gen.manual_seed(lay.cfg.seed)
    wbuf = torch.empty(cold_bytes, dtype=torch.uint8, device=device)
    w16 = wbuf.view(torch.bfloat16)
    for o in range(0, w16.numel(), 1 << 26):
        c = min(1 << 26, w16.numel() - o)
        w16[o:o + c] = (torch.randn(c, device=device, generator=gen) * 0.02).bfloat16()
    rows_of = lambda n: sum(n) if isinstance(n, tuple) else n
    kmax = max(k for (_, k, _, _) in shapes)
    nmax = max(rows_of(n) for (n, _, _, _) in shapes)
    mmax = max(m for (_, _, _, m) in shapes)
    # two activation buffers: a launch that is the first over its activations (another kernel has just written them in a real
    # step) takes the other one, so that only the launches that follow it may request their activations early (tgp_k_gemm_chain)
    A2 = [torch.randn((mmax, kmax), device=device, generator=gen).bfloat16() for _ in range(2)]
    new_acts = gemm_shapes_of_step.new_acts
    tb.k_gemm_chain(True)
    Cbuf = torch.zeros((mmax, nmax), dtype=torch.float32, device=device)
    stream = torch.cuda.Stream(device=device)
    off = 0

    kernel_of = {}

    def run_all(st, only=None):
        nonlocal off
        which = 0
        for idx, (n, K, res, m) in enumerate(shapes):
            if idx in new_acts:
                which ^= 1
            A = A2[which]
            if only is not None and (n, K, res, m) != only:
                continue
            nb = (rows_of(n) * K * 2 + 511) // 512 * 512
            if off + nb > cold_bytes:
                off = 0
            if isinstance(n, tuple):
                starts = [sum(n[:i]) for i in range(len(n))]
                tb.k_gemm_group(A, [wbuf.data_ptr() + off + r0 * K * 2 for r0 in starts], [Cbuf.data_ptr() + r0 * 4 for r0 in starts],
                                m, list(n), K, [nmax] * len(n), res, st)
            else:
                tb.k_gemm(A, wbuf.data_ptr() + off, Cbuf, m, n, K, nmax, 0, res, st)
            kernel_of[(n, K, res, m)] = tb.k_gemm_last_kernel()
            off += nb

    def graph_of(only=None, passes=4):
        """The launch sequence captured in a CUDA graph (several passes at successive cold offsets), so that the
        replay is paced by the device, not by Python."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(passes):
                run_all(torch.cuda.current_stream(), only)
        return g, passes

    for _ in range(3):
        run_all(stream)
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    def bounded(g, want_s):
        """One untimed-for-the-result replay measures a replay's length; then as many replays as fill want_s seconds are
        timed (want_s == 0: `reps` replays, but no more than fit in 4 s - a deep model's step has thousands of launches)."""
        with torch.cuda.stream(stream):
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
            one = max(1e-6, e0.elapsed_time(e1) * 1e-3)
            n = max(1, min(200000, int(np.ceil(want_s / one)))) if want_s > 0 else max(1, min(reps, int(4.0 / one)))
            e0.record(stream)
            for _ in range(n):
                g.replay()
            e1.record(stream)
        stream.synchronize()
        return n, e0.elapsed_time(e1) * 1e-3

    g, passes = graph_of()
    n_rep, total_s = bounded(g, min_seconds)
    kernel_loop.last = {"reps": n_rep, "passes": passes, "seconds": total_s}
    sec = total_s / (n_rep * passes * len(shapes))
    bytes_per = sum(2 * m * K + 2 * K * rows_of(n) + 4 * m * rows_of(n) * (2 if res else 1) for (n, K, res, m) in shapes) / len(shapes)
    flops_per = sum(2 * m * K * rows_of(n) for (n, K, res, m) in shapes) / len(shapes)
    table = {}
    for sh in sorted(set(shapes), key=lambda q: (rows_of(q[0]),) + tuple(q[1:])):
        cnt = shapes.count(sh)
        g, passes = graph_of(only=sh)
        n_sh, t_sh = bounded(g, min(0.3, min_seconds))
        t = t_sh / (n_sh * passes * cnt)
        n, K, res, m = sh
        nr = rows_of(n)
        b = 2 * m * K + 2 * K * nr + 4 * m * nr * (2 if res else 1)
        name = "+".join(str(x) for x in n) if isinstance(n, tuple) else str(n)
        table[f"n={name} K={K} M={m} res={res}"] = {"kernel": kernel_of.get(sh, "?"), "launches_per_step": cnt, "us": round(t * 1e6, 2),
                                                      "GBps": round(b / t / 1e9, 1), "TFLOPs": round(2 * m * K * nr / t / 1e12, 2)}
    tb.k_gemm_chain(False)
    return sec, bytes_per, flops_per, len(shapes), table


def attention_loop(cfg, reps, device):
    """Times the causal prefill attention of one layer at the workload's shape (B sequences of S queries, KV in the
    engine's tile layout), once per kernel: the tcgen05 kernel, the mma.sync kernel, and the automatic choice.
    Flops are the causal ones, 4 * B * Hq * Dh * S (S + 1) / 2.  Q, K, V: seeded normal values."""
    import torch
    from paper_2609_06172_b200 import binding as tb
    from paper_2609_06172_b200.session import model_cfg
    mc = model_cfg(cfg)
    B, S = cfg.B, cfg.S
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed)
    n = B * cfg.Hkv * cfg.TK * cfg.Dh
    n_tiles = (S + cfg.TK - 1) // cfg.TK
    kt = [torch.randn(n, device=device, generator=g).bfloat16() for _ in range(n_tiles)]
    vt = [torch.randn(n, device=device, generator=g).bfloat16() for _ in range(n_tiles)]
    qb = torch.randn(B * S, cfg.Hq * cfg.Dh, device=device, generator=g).bfloat16()
    ob = torch.zeros(B * S, cfg.Hq * cfg.Dh, dtype=torch.bfloat16, device=device)
    flops = 4 * B * cfg.Hq * cfg.Dh * S * (S + 1) / 2
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)         # larger than L2: written between timed launches
    out = {}
    for name, impl in (("tcgen05", 3), ("mma_sync", 2), ("auto", 0)):
        tb.k_attn_select(impl)
        for _ in range(3):
            tb.k_attn(qb, kt, vt, ob, mc, B, S, 0, None)
        torch.cuda.synchronize()
        ms = 0.0
        for _ in range(reps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            tb.k_attn(qb, kt, vt, ob, mc, B, S, 0, None)
            e1.record()
            torch.cuda.synchronize()
            ms += e0.elapsed_time(e1)
        t = ms * 1e-3 / reps
        out[name] = {"us": round(t * 1e6, 1), "TFLOPs": round(flops / t / 1e12, 1)}
    tb.k_attn_select(0)
    out["status"] = tb.k_attn_status()
    # decode: one query per sequence over the same S keys (KV bytes read once: 2 * B * Hkv * S * Dh * 2), per kernel
    q1 = qb[:B].contiguous()
    o1 = torch.zeros(B, cfg.Hq * cfg.Dh, dtype=torch.bfloat16, device=device)
    scratch = torch.empty(tb.k_attn_scratch_bytes(mc) // 4, dtype=torch.float32, device=device)
    kv_bytes = 2 * B * cfg.Hkv * S * cfg.Dh * 2
    for name, impl in (("decode_mma", 2), ("decode_cuda_core", 1), ("decode", 0)):
        tb.k_attn_decode_select(impl)
        for _ in range(3):
            tb.k_attn(q1, kt, vt, o1, mc, B, 1, S - 1, scratch)
        torch.cuda.synchronize()
        ms = 0.0
        for _ in range(reps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            tb.k_attn(q1, kt, vt, o1, mc, B, 1, S - 1, scratch)
            e1.record()
            torch.cuda.synchronize()
            ms += e0.elapsed_time(e1)
        t = ms * 1e-3 / reps
        out[name] = {"us": round(t * 1e6, 1), "GBps": round(kv_bytes / t / 1e9, 1), "kv_bytes": kv_bytes}
    tb.k_attn_decode_select(0)
    return out, flops


def whole_job_rate(units_per_rank, ms_local, dist=None, device=None):
    """Replicas: every rank processed `units_per_rank` units in `ms_local`; the job's rate is all units over the
    slowest rank's time.  The only collective is this MAX reduction of the timing (none on the data path)."""
    world, ms = 1, float(ms_local)
    if dist is not None and dist.is_initialized():
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms, world = float(t.item()), dist.get_world_size()
    return world * units_per_rank / (ms * 1e-3), ms, world


def oracle_sample(cfg, lay):
    """Bounded sample for timing the oracle: about 5e11 flops of prefill (at most 128 prompt tokens per sequence)
    plus up to 4 decode steps, at full widths and depth."""
    params = lay.weight_bytes // 2
    return int(max(4, min(128, cfg.S, 5e11 / (2 * params * cfg.B)))), min(cfg.T, 4)


def run_reference(args, cfg, lay, full_T=None):
    """The CPU oracle, as it stands, through the bench contract: every step is a bounded sample of the workload named in
    `config` (full widths and depth, a prefix of the prompt and of the decode steps), on the host cores of rank 0."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    pool = np.empty(lay.pool_bytes, dtype=np.uint8)
    filled = False
    if lay.pool_bytes > (1 << 30):
        # seeded inputs of a multi-gigabyte pool: the same generator evaluated on a GPU when one is there (bit-identical
        # to the numpy generator, tested); the oracle's arithmetic below runs on the host cores either way
        try:
            import torch
            if torch.cuda.is_available():
                si.fill_pool_torch(lay, torch.from_numpy(pool), device="cuda:0")
                filled = True
        except Exception:
            filled = False
    if not filled:
        si.fill_pool(lay, pool)
    om = make_oracle(lay, oracle_weights_from_pool(lay, pool))
    del pool
    sS, sT = oracle_sample(cfg, lay)
    cores = len(os.sched_getaffinity(0))
    for _ in range(args.warmup):
        time_oracle(lay, om, min(16, sS), 1)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(lay, om, sS, sT)
    dt = time.perf_counter() - t0
    val = cfg.B * (sS + sT) * args.steps / dt
    sample = f"prefill of the first {sS} prompt tokens + {sT} decode steps per step (full widths and depth)"
    print(json.dumps({"impl": "reference", "metric": "tokens_per_s", "value": val, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
                      "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
                      "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": config_dict(cfg, lay, full_T, int(os.environ.get("WORLD_SIZE", "1"))), "sample": sample,
                      "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
                      "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# decode steps per timed pass where the configuration's own count would make a pass run for tens of seconds (per-step
# rates do not depend on the count; the workload string names what ran): headline pass, one-pass summary
DECODE_PER_PASS = {3: 32, 4: 4, 5: 8}
DECODE_PER_SUMMARY = {3: 16, 4: 2, 5: 4}
ALIAS_LAYERS = {4: 40}          # the 70B shape's 152 GB pool cannot be page-locked on a 206 GB host: 40 physical layers, each mapped twice
HEADLINE_CONFIG = 3


def workload_name(cfg, lay, full_T=None):
    dec = f"{cfg.T}" if full_T in (None, cfg.T) else f"{cfg.T} of {full_T}"
    return (f"{cfg.name}: L={cfg.L} d={cfg.d} Hq/Hkv={cfg.Hq}/{cfg.Hkv} F={cfg.F} V={cfg.V} B={cfg.B} prompt={cfg.S} decode={dec} "
            f"pool={lay.pool_bytes} budget={lay.budget}")


def config_dict(cfg, lay, full_T, world=1, graph=False):
    return {"workload": workload_name(cfg, lay, full_T), "l2": f"inputs larger than L2: every decode step streams the {lay.pool_bytes / 1e9:.1f} GB pool",
            "step": "prefill + %d decode steps from a cold arena" % cfg.T + (", replayed as one CUDA graph" if graph else ""),
            "tokens_per_step": cfg.B * (cfg.S + cfg.T), "parallelism": "replicas" if world > 1 else "single"}


def lower_bound_bytes(ops, lay):
    """Per step: bytes that must cross the link whatever the schedule = accessed pool bytes - budget (all of them for
    the cold first step); a tensor counts once per step, at its largest access of the step (whole if any access
    touches half of it or more)."""
    step_of = {}
    for o in ops:
        d = step_of.setdefault(o[0], {})
        for (t, mode, touched) in o[6]:
            b = lay.tensors[t].size if touched * 2 >= lay.tensors[t].size else touched
            d[t] = max(d.get(t, 0), b)
    return {k: max(0, sum(d.values()) - (lay.budget if k else 0)) for k, d in step_of.items()}


def step_roofline(ops, totals, lay, t_meas, step_ms):
    """Slowest of compute, HBM and link per step, summed over the steps of a pass: (i) with the plan's link bytes,
    (ii) with the lower bound on them."""
    nsteps = len(totals)
    Fs, Hs = [0] * nsteps, [0] * nsteps
    for o in ops:
        Fs[o[0]] += o[4]
        Hs[o[0]] += o[5]
    lb = lower_bound_bytes(ops, lay)
    t_roof = t_lb = 0.0
    bound_of = []
    for k in range(nsteps):
        cands = {"tensor": Fs[k] / MACHINE["peak_flops"], "hbm": (Hs[k] + int(totals[k][0])) / MACHINE["hbm_Bps"],
                 "link": (int(totals[k][0]) + int(totals[k][2])) / MACHINE["h2d_Bps"], "link_d2h": int(totals[k][1]) / MACHINE["d2h_Bps"]}
        bound_of.append(max(cands, key=cands.get))
        t_roof += max(cands.values())
        t_lb += max(cands["tensor"], cands["hbm"], lb.get(k, 0) / MACHINE["h2d_Bps"])
    L_plan = int(totals[:, 0].sum() + totals[:, 2].sum())
    return {"bound": {"prefill": bound_of[0], "decode": max(set(bound_of[1:]), key=bound_of[1:].count) if nsteps > 1 else None},
            "t_roof_s_plan_bytes": t_roof, "t_roof_s_lower_bound": t_lb, "t_measured_s": t_meas,
            "frac_plan_bytes": t_roof / t_meas, "frac_lower_bound": t_lb / t_meas,
            "prefill": {"t_roof_s": max(Fs[0] / MACHINE["peak_flops"], (int(totals[0][0]) + int(totals[0][2])) / MACHINE["h2d_Bps"]),
                        "t_measured_s": step_ms[0] * 1e-3 if step_ms else None},
            "link_gbs_achieved": L_plan / t_meas / 1e9, "link_gbs_peak": MACHINE["h2d_Bps"] / 1e9,
            "h2d_bytes": int(totals[:, 0].sum()), "d2h_bytes": int(totals[:, 1].sum()), "zero_copy_bytes": int(totals[:, 2].sum()),
            "flops": sum(Fs), "hbm_bytes": sum(Hs) + int(totals[:, 0].sum())}


def other_config_summaries(args, budget_s):
    """One-pass summaries of the other configurations, each in a process of its own (its host pool is released when it
    exits) under a time limit; what does not fit the remaining budget is reported as skipped, never silently dropped."""
    out = {}
    t_end = time.monotonic() + budget_s
    for c in (1, 2, 5, 4):
        if c == args.config:
            continue
        left = t_end - time.monotonic()
        if left < 60:
            out[str(c)] = {"skipped": "time budget of this run spent"}
            continue
        for key, extra in ((str(c), []),) + ((("1_graph", ["--graph"]),) if c == 1 else ()):      # the tiny configuration also as one CUDA graph per pass
            cmd = [sys.executable, os.path.abspath(__file__), "--config", str(c), "--summary"] + extra
            t0 = time.monotonic()
            try:
                r = subprocess.run(cmd, capture_output=True, text=True, timeout=min(left, 600))
                line = [l for l in r.stdout.splitlines() if l.startswith("{")]
                out[key] = json.loads(line[-1]) if r.returncode == 0 and line else {"failed": f"rc {r.returncode}", "stderr_tail": r.stderr[-400:]}
            except subprocess.TimeoutExpired:
                out[key] = {"failed": "time limit"}
            out[key]["wall_s"] = round(time.monotonic() - t0, 1)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="tgp")
    ap.add_argument("--config", type=int, default=HEADLINE_CONFIG)
    ap.add_argument("--decode", type=int, default=None, help="decode steps per pass (default: the configuration's, bounded for configs 3-5)")
    ap.add_argument("--summary", action="store_true", help="one warm-up pass and one timed pass, compact output (what the headline run collects for the other configurations)")
    ap.add_argument("--no-configs", action="store_true", help="skip the one-pass summaries of the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-uvm", action="store_true", help="skip the demand-paged managed-memory baseline")
    ap.add_argument("--kernel-loop", choices=["decode", "prefill", "attention"], default=None,
                    help="only run the back-to-back weight-product loop of one step (small, for ncu captures)")
    ap.add_argument("--planned-mix", action="store_true",
                    help="with --kernel-loop decode/prefill: the launch list of the planned run at the configuration's budget (blocks staged "
                         "through the ring end their launch) instead of every block resident")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--alias-layers", type=int, default=None, help="host pool with this many physical layers: layers l and l + N share host pages (for pools larger than the host can page-lock)")
    ap.add_argument("--unseen-prompts", action="store_true", help="MoE: time prompts of another seed than the profile pass saw")
    ap.add_argument("--seq", type=int, default=None, help="with --kernel-loop attention: prompt length instead of the configuration's")
    ap.add_argument("--graph", action="store_true", help="replay the whole planned run as one CUDA graph (dense models; for host-bound tiny steps)")
    ap.add_argument("--layers", type=int, default=None, help="run the shape at reduced depth; a byte budget is scaled in proportion")
    ap.add_argument("--cap-mib", type=float, default=None, help="sub-range cap in MiB (default: the input recipe's rule)")
    ap.add_argument("--bits", type=int, default=15, help="policy bits: 1 affinity/pins, 2 roofline selectivity, 4 zero-copy, 8 windowed pin reservation")
    ap.add_argument("--budget-frac", type=float, default=None, help="device budget as a fraction of the pool (oversubscription sweep)")
    args = ap.parse_args()
    cfg = si.CONFIGS[args.config]
    full_T = cfg.T
    if args.decode is not None:
        cfg = replace(cfg, T=args.decode)
    elif args.config in DECODE_PER_PASS and not args.kernel_loop:
        cfg = replace(cfg, T=min(cfg.T, (DECODE_PER_SUMMARY if args.summary else DECODE_PER_PASS)[args.config]))
    if args.alias_layers is None and args.config in ALIAS_LAYERS and args.layers is None and args.impl != "reference" and not args.kernel_loop:
        args.alias_layers = ALIAS_LAYERS[args.config]
    if args.summary:
        args.steps, args.warmup, args.no_configs, args.no_cpu_baseline = (20, 5, True, True) if args.config == 1 else (1, 1, True, True)
        args.no_uvm = args.no_uvm or args.config != 2
    budget = None
    if args.layers is not None and args.layers != cfg.L:
        full = si.build_layout(cfg)
        cfg2 = replace(cfg, L=args.layers, name=f"{cfg.name}_L{args.layers}")
        budget = int(full.budget * si.build_layout(cfg2, budget=1 << 40).pool_bytes / full.pool_bytes) // 512 * 512
        cfg = cfg2
    cap = int(args.cap_mib * (1 << 20)) if args.cap_mib else None
    lay = si.build_layout(cfg, budget=budget, cap=cap)
    if args.budget_frac is not None:
        lay = si.build_layout(cfg, budget=int(lay.pool_bytes * args.budget_frac) // 512 * 512, cap=cap)
    if args.impl == "reference":
        return run_reference(args, cfg, lay, full_T)

    if args.kernel_loop:
        import torch
        from paper_2609_06172_b200 import binding as tb
        tb.lib()
        if args.kernel_loop == "attention":
            if args.seq:
                cfg = replace(cfg, S=args.seq)
            table, flops = attention_loop(cfg, args.reps, torch.device("cuda:0"))
            print(json.dumps({"kernel_loop": "attention", "config": cfg.name, "B": cfg.B, "S": cfg.S, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "Dh": cfg.Dh,
                              "TK": cfg.TK, "causal_flops": flops, "L2_flushed_between_launches": True, "kernels": table}))
            return
        M = cfg.B * (cfg.S if args.kernel_loop == "prefill" else 1)
        pinned = None
        if args.planned_mix and not cfg.E:
            # the launch list of the planned, oversubscribed run: planned on the host (no pool needed), pins read from the plan
            from paper_2609_06172_b200.session import Session
            ps = Session(lay, MACHINE)
            pb = ps.plan(bits=args.bits)["pins"]
            pinned = {struct.unpack_from("<IQ", pb, 12 * k)[0] for k in range((len(pb) - 16) // 12)}
            ps.close()
        sec, b, f, nl, table = kernel_loop(lay, M, args.reps, torch.device("cuda:0"), min_seconds=0.0, pinned=pinned)
        print(json.dumps({"kernel_loop": args.kernel_loop, "M": M, "avg_us": sec * 1e6, "GBps": b / sec / 1e9, "TFLOPs": f / sec / 1e12,
                          "launches_per_step": nl, "launch_list": "planned run" if pinned is not None else "every block resident",
                          "timed": kernel_loop.last, "shapes": table}))
        return

    t_start = time.monotonic()
    import torch
    from paper_2609_06172_b200 import binding as tb
    from paper_2609_06172_b200.runner import Runner, pinned_pool
    from paper_2609_06172_b200.session import Session
    tb.lib()                                                     # fails loudly when the CUDA library is missing
    rank, world, local = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    aliased = None
    if args.alias_layers:
        # more weights than this host can page-lock: layers l and l + alias_layers share physical host pages (same
        # virtual layout, same bytes over the link, same arithmetic; logits are those of a model with repeated layers)
        from paper_2609_06172_b200.runner import AliasedPool
        aliased = AliasedPool(lay, args.alias_layers)
        pool = torch.from_numpy(aliased.numpy())
        aliased.page_lock()
    else:
        pool = pinned_pool(lay.pool_bytes)
    si.fill_pool_torch(lay, pool, device=dev)
    bias = si.router_bias(cfg) if cfg.E else None
    s = Session(lay, MACHINE, pool_base=pool.data_ptr(), pool_flags=tb.POOL_PINNED, router_bias=bias)
    profile_s = None
    if cfg.E:
        # MoE: one profile pass with every expert traced records which experts each step really uses
        s.plan(expert_counts=np.ones((1 + cfg.T, cfg.L, cfg.E), dtype=np.uint32), bits=args.bits)
        r = Runner(s, cfg.B * cfg.S, device=str(dev))
        t0 = time.perf_counter()
        r.generate(si.prompt_tokens(cfg), cfg.T, keep_logits=False)
        profile_s = time.perf_counter() - t0
        counts = s.ctx.expert_counts(cfg.L, cfg.E)
        blobs = s.plan(expert_counts=counts, bits=args.bits)
    else:
        blobs = s.plan(bits=args.bits)
        r = Runner(s, cfg.B * cfg.S, device=str(dev))
    totals = np.frombuffer(blobs["totals"], dtype="<u8").reshape(-1, 4)
    ops = s.ctx.trace_ops()
    # --unseen-prompts (MoE): the timed passes run prompts the profile pass never saw, so the plan's expert sets are a
    # prediction; an expert the router picks outside its step's set is fetched synchronously and counted
    run_cfg = replace(cfg, seed=cfg.seed ^ 0x5EED) if args.unseen_prompts else cfg
    prompt_pinned = torch.from_numpy(si.prompt_tokens(run_cfg)).pin_memory()
    tok_pinned = torch.empty((cfg.B, 1), dtype=torch.int32).pin_memory()
    logits_host = torch.empty((cfg.B, cfg.V), dtype=torch.float32).pin_memory()
    T = cfg.T

    use_graph = args.graph and not cfg.E

    def one_pass(e2e=False):
        if use_graph and not e2e:
            r.replay()
            return
        r.reset()
        r.step(tb.PREFILL, prompt_pinned.numpy(), cfg.S)
        for t in range(T):
            if e2e:
                with torch.cuda.stream(r.compute):
                    tok_pinned.copy_(r.argmax.view(cfg.B, 1), non_blocking=True)
                r.compute.synchronize()
                r.step(tb.DECODE, tok_pinned.numpy(), 1)
            else:
                r.step(tb.DECODE, None, 1)
        if e2e:
            with torch.cuda.stream(r.compute):
                logits_host.copy_(r.logits, non_blocking=True)
                tok_pinned.copy_(r.argmax.view(cfg.B, 1), non_blocking=True)
            r.compute.synchronize()

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(n, e2e):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(r.compute)
        for _ in range(n):
            one_pass(e2e)
        r.sync()                                                 # every stream of the device, the library's write-back stream included
        ev1.record(r.compute)
        r.sync()
        barrier()
        return whole_job_rate(1, ev0.elapsed_time(ev1), dist, dev)[1]

    if use_graph:
        r.reset()
        r.step(tb.PREFILL, prompt_pinned.numpy(), cfg.S)             # one plain pass first: kernel attributes are set up outside capture
        for t in range(T):
            r.step(tb.DECODE, None, 1)
        r.sync()
        r.capture_run(prompt_pinned, T)
    for _ in range(args.warmup):
        one_pass(False)
    r.sync()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms = timed(args.steps, False)
    clocks = sampler.stop() if rank == 0 else None
    if use_graph:
        r.sync()
        r.reset()
    ms_e2e = None
    # the end-to-end passes repeat the timed ones with the host copies inside: at seconds per pass five of them are enough
    # (the whole default run, the other configurations' summaries included, is meant to stay within about eight minutes)
    n_e2e = args.steps if ms / args.steps < 2000.0 else min(args.steps, 5)
    if not args.summary:
        one_pass(True)
        ms_e2e = timed(n_e2e, True)
    tokens_per_pass = cfg.B * (cfg.S + T)
    value = world * tokens_per_pass * args.steps / (ms * 1e-3)
    e2e_value = world * tokens_per_pass * n_e2e / (ms_e2e * 1e-3) if ms_e2e else None

    # ---- per-phase timing, launches and the live per-kernel roofline: one extra pass with op timestamps -----------
    # (step times from a pass without op timestamps: the event brackets around every op keep consecutive launches from
    # overlapping, which a step of a few milliseconds would feel)
    r.reset()
    launches = mismatches = 0
    step_ms = []
    for k in range(1 + T):
        st = r.step(tb.PREFILL if k == 0 else tb.DECODE, prompt_pinned.numpy() if k == 0 else None, cfg.S if k == 0 else 1, want_stats=True)
        launches += st.n_launches
        mismatches += st.n_mismatch
        step_ms.append(st.step_ms)
    r.reset()
    s.ctx.set_op_timing(True)
    kind_ms, kind_bytes, kind_flops, kind_n = {}, {}, {}, {}
    for k in range(1 + T):
        st = r.step(tb.PREFILL if k == 0 else tb.DECODE, prompt_pinned.numpy() if k == 0 else None, cfg.S if k == 0 else 1, want_stats=True)
        first, tms = s.ctx.op_times()
        phase = "prefill" if k == 0 else "decode"
        for j, t in enumerate(tms):
            o = ops[first + j]
            key = (phase, OP_NAMES[o[3]])
            kind_ms[key] = kind_ms.get(key, 0.0) + float(t)
            kind_bytes[key] = kind_bytes.get(key, 0) + o[5]
            kind_flops[key] = kind_flops.get(key, 0) + o[4]
            kind_n[key] = kind_n.get(key, 0) + 1
    s.ctx.set_op_timing(False)
    r.sync()
    moe_prediction = None
    if cfg.E:
        ran = s.ctx.expert_counts(cfg.L, cfg.E)
        n = min(len(ran), len(counts))
        planned, used = np.asarray(counts[:n]) > 0, np.asarray(ran[:n]) > 0
        moe_prediction = {"expert_slots_planned": int(planned.sum()), "planned_but_unused": int((planned & ~used).sum()),
                          "used_but_unplanned": int((~planned & used).sum()), "slots": int(planned.size)}
        # realised popularity: share of routed (token, slot) pairs by the expert's rank in its layer's bias, beside the
        # Zipf law the bias encodes for the first choice (top-2 routing flattens it: the second choice is someone else)
        order = np.argsort(-np.asarray(bias), axis=1)                                   # [L, E]: experts by falling bias
        by_rank = np.zeros(cfg.E)
        tot = np.asarray(ran[:n], dtype=np.float64).sum(axis=0)                          # [L, E]
        for l in range(cfg.L):
            by_rank += tot[l][order[l]]
        zipf = np.array([r_ ** (-cfg.zipf_s) for r_ in range(1, cfg.E + 1)])
        moe_prediction["routed_share_by_bias_rank"] = [round(float(x), 4) for x in by_rank / max(1.0, by_rank.sum())]
        moe_prediction["zipf_first_choice"] = [round(float(x), 4) for x in zipf / zipf.sum()]

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    t_meas = ms * 1e-3 / args.steps
    step_roof = step_roofline(ops, totals, lay, t_meas, step_ms)
    host_pool = ({"aliased_physical_layers": args.alias_layers, "physical_bytes": aliased.phys_bytes, "virtual_bytes": lay.pool_bytes,
                  "note": "layers l and l + %d share host pages: link bytes, schedule and arithmetic are the full model's; throughput only" % args.alias_layers}
                 if aliased else "pinned, one physical page per byte")
    prefill_tok_s = cfg.B * cfg.S / (step_ms[0] * 1e-3)
    decode_tok_s = cfg.B * T / (sum(step_ms[1:]) * 1e-3) if T else None
    if args.summary:
        out = {"config": args.config, "workload": workload_name(cfg, lay, full_T), "passes_timed": args.steps, "tokens_per_s": value,
               "prefill_tok_s": prefill_tok_s, "decode_tok_s": decode_tok_s, "ms_per_pass": ms / args.steps,
               "step_roofline": {k: step_roof[k] for k in ("bound", "frac_plan_bytes", "frac_lower_bound", "link_gbs_achieved", "link_gbs_peak", "t_measured_s")},
               "host_pool": host_pool, "gpu_launches": launches, "clocks": clocks, "trace_mismatches": mismatches, "graph": bool(use_graph),
               "kernels_ms": {f"{k[0]}:{k[1]}": round(v, 3) for k, v in sorted(kind_ms.items())}}
        if not args.no_uvm:
            out["uvm"] = uvm_runs(args, cfg, lay, dev, pool, r, s, step_ms, T, only_demand=True)
        print(json.dumps(out))
        return
    peaks = measured_peaks()
    # dominant kernel by device time in the pass; its launch duration is measured in a dedicated region: the same
    # launches back to back on one stream over cold inputs (in-step event brackets of microsecond kernels also
    # measure the wake-up of a stream that was waiting on a copy, see kernels[*].ms)
    dom = max(kind_ms, key=lambda k: kind_ms[k])
    if dom[1] == "gemm":
        Mk = cfg.B * (cfg.S if dom[0] == "prefill" else 1)
        pb = s.ctx.plan_blobs()["pins"]
        pinned = {struct.unpack_from("<IQ", pb, 12 * k)[0] for k in range((len(pb) - 16) // 12)}
        sec, bpl, fpl, nl, table = kernel_loop(lay, Mk, args.reps, dev, pinned=pinned)
        timed_mix = dict(kernel_loop.last)
        # the same products with every block resident (what tgp_step launches when the budget holds the pool: all pieces of
        # a matrix in one launch), for comparison with the mix of the oversubscribed run
        sec_res, bpl_res, _, nl_res, _ = kernel_loop(lay, Mk, args.reps, dev, min_seconds=0.5, pinned=None)
        kernel_loop.last = timed_mix
        if dom[0] == "prefill" and fpl / MACHINE["peak_flops"] > bpl / MACHINE["hbm_Bps"]:
            ach = fpl / sec / 1e12
            # the loop below replays the step's launches for seconds under the power cap: the matching denominator is the
            # sustained cuBLAS figure (the burst figure is for a kernel timed alone for a millisecond)
            loop_s = kernel_loop.last["seconds"]
            pk = peaks["bf16_sustained"] if (loop_s > 1.0 and peaks.get("bf16_sustained")) else peaks["bf16_tflops"]
            roof = {"bound": "tensor", "achieved": ach, "peak": pk, "unit": "TFLOP/s", "frac": ach / pk,
                    "peak_kind": "sustained cuBLAS bf16 (timed loop of %.1f s)" % loop_s if pk != peaks["bf16_tflops"] else "burst cuBLAS bf16",
                    "frac_of_burst_peak": ach / peaks["bf16_tflops"]}
        else:
            ach = bpl / sec / 1e9
            roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                    "all_blocks_resident": {"launches_per_step": nl_res, "avg_us": sec_res * 1e6, "achieved": bpl_res / sec_res / 1e9,
                                            "frac": bpl_res / sec_res / 1e9 / peaks["hbm_gbs"],
                                            "note": "the same products as tgp_step launches them when no block is staged through the ring (budget >= pool)"}}
        # the kernels that ran, as the library reports them per launch (its choice depends on M, n, K), heaviest first
        by_kernel = {}
        for v in table.values():
            by_kernel[v["kernel"]] = by_kernel.get(v["kernel"], 0.0) + v["us"] * v["launches_per_step"]
        names = sorted(by_kernel, key=by_kernel.get, reverse=True)
        roof.update({"kernel": f"weight-block product ({dom[0]}, M={Mk}): " + " + ".join(names),
                     "kernel_time_share": {k: round(by_kernel[k] / sum(by_kernel.values()), 3) for k in names},
                     "launches": nl * (T if dom[0] == "decode" else 1), "avg_us": sec * 1e6, "algorithmic_per_launch": fpl if roof["bound"] == "tensor" else bpl,
                     "timing": f"CUDA-graph replay of the {nl} weight-block launches of one step of the timed run (blocks the plan pins share launches, a block staged through the ring ends its launch), {kernel_loop.last['reps']} x {kernel_loop.last['passes']} passes back to back ({kernel_loop.last['seconds']:.2f} s), random operands, cold inputs cycling through 1 GiB, CUDA events on the launch stream",
                     "in_step_avg_us": kind_ms[dom] / (nl * (T if dom[0] == "decode" else 1)) * 1e3, "shapes": table})
    else:
        ach = kind_bytes[dom] / (kind_ms[dom] * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "kernel": f"{dom[1]} ({dom[0]})", "launches": kind_n[dom], "avg_us": kind_ms[dom] / kind_n[dom] * 1e3,
                "algorithmic_per_launch": kind_bytes[dom] / kind_n[dom], "timing": "in-step CUDA events per op"}
    roof.update({"peak_source": peaks["source"], "traffic": None})
    prof = os.path.join(ROOT, "profiles", "traffic.txt")          # DRAM bytes per launch from the committed ncu summaries
    if os.path.exists(prof):
        for line in open(prof):
            f = line.split(None, 2)
            if f and f[0] == f"{dom[1]}_{dom[0]}_cfg{args.config}":
                roof["traffic"] = float(f[1])
                roof["traffic_source"] = "profiles/traffic.txt: " + (f[2].strip().strip('"') if len(f) > 2 else "ncu capture")
    # the paper's motivation experiment (Section III-B) on this workload, analytically: a prefetcher that sees only
    # allocator segments (20 MiB, the large-block size of PyTorch's caching allocator) and prefetches every segment
    # an op's tensors overlap moves this many useless bytes per useful byte
    SEG = 20 << 20
    useful = useless = 0
    for o in ops:
        segs = set()
        for (t, mode, touched) in o[6]:
            tt = lay.tensors[t]
            segs.update(range(tt.pool_off // SEG, (tt.pool_off + tt.size - 1) // SEG + 1))
            useful += touched
        useless += len(segs) * SEG
    object_level = {"segment_bytes": SEG, "useless_over_useful": (useless - useful) / max(1, useful), "kind": "analytic, from the trace"}
    L_d2h = int(totals[:, 1].sum())
    out = {"metric": "tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
           "data": "synthetic", "config": config_dict(cfg, lay, full_T, world, use_graph),
           "prefill_tok_s": prefill_tok_s, "decode_tok_s": decode_tok_s,
           "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": int(totals[:, 0].sum()) + cfg.B * (cfg.S + T) * 4,
                   "d2h_bytes_per_step": L_d2h + cfg.B * (T + 1) * 4 + cfg.B * cfg.V * 4, "passes_timed": n_e2e},
           "object_level_prefetch": object_level, "policy_bits": args.bits, "trace_mismatches": mismatches, "moe_profile_pass_s": profile_s, "unseen_prompts": bool(args.unseen_prompts),
           "host_pool": host_pool, "moe_prediction": moe_prediction,
           "gpu_launches": launches * args.steps, "clocks": clocks, "roofline": roof, "step_roofline": step_roof,
           "kernels": {f"{k[0]}:{k[1]}": {"ms": round(v, 3), "ops": kind_n[k], "GBps": round(kind_bytes[k] / (v * 1e-3) / 1e9, 1),
                                           "TFLOPs": round(kind_flops[k] / (v * 1e-3) / 1e12, 2)} for k, v in sorted(kind_ms.items())}}
    pool_np = pool.numpy()
    if not args.no_cpu_baseline and world == 1:
        # the oracle, timed on the host cores on a bounded sample of this workload - and, on the same sample, compared
        # with the GPU path's logits (teacher-forced, free-running: no lockstep), so that the line carries a live parity figure
        om = make_oracle(lay, oracle_weights_from_pool(lay, pool_np))
        sS, sT = oracle_sample(cfg, lay)
        sample_prompt = si.prompt_tokens(cfg)[:, :sS]
        om.generate(sample_prompt[:, :min(16, sS)], 1)
        t0 = time.perf_counter()
        ref_logits, ref_toks = om.generate(sample_prompt, sT)
        dt = time.perf_counter() - t0
        val = cfg.B * (sS + sT) / dt
        out["cpu_baseline"] = {"value": val, "unit": "tokens/s", "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                               "sample": f"prefill of the first {sS} prompt tokens + {sT} decode steps, float32 accumulate ({dt:.1f} s)"}
        if not cfg.E:
            try:
                s.plan(S=sS, T=sT, bits=args.bits)
                got, _ = r.generate(sample_prompt, sT, forced=ref_toks)
                errs = [np.abs(a - b) for a, b in zip(got, ref_logits)]
                out["parity_sample"] = {"sample": f"the CPU baseline's sample (full widths and depth, {cfg.B} x {sS} prompt tokens + {sT} decode steps, the oracle's tokens fed to both)",
                                        "max_abs_logit_error": float(max(e.max() for e in errs)),
                                        "mean_rel_logit_error": float(max(e.mean() / np.abs(b).mean() for e, b in zip(errs, ref_logits))),
                                        "argmax_agreement": float(np.mean([np.mean(np.argmax(a, -1) == np.argmax(b, -1)) for a, b in zip(got, ref_logits)])),
                                        "stated_tolerance": {"max_abs": 3e-2, "mean_rel": 1e-2},
                                        "note": "free-running comparison against the float32 oracle: at this depth bf16 rounding flips decorrelate any two summation orders (tests/golden/precision_floor.txt); the element-by-element criterion is the lockstep test"}
            except Exception as ex:
                out["parity_sample"] = f"not run: {type(ex).__name__}: {ex}"
        del om, ref_logits
    if not args.no_uvm and world == 1:                 # the baselines are single-GPU measurements: reported at N = 1 only
        uvm = uvm_runs(args, cfg, lay, dev, pool, r, s, step_ms, T, only_demand=False)
        out["uvm"] = uvm
        mo = uvm.get("managed_object") if isinstance(uvm, dict) else None
        if mo and mo.get("asked_bytes_per_decode_step"):
            # the same experiment run for real: the managed pool with the segment-granular prefetcher one op ahead
            touched = sum(a[2] for o in ops if o[0] >= 1 for a in o[6]) / max(1, T)
            object_level["measured"] = {"decode_tok_s": mo["decode_tok_s"], "asked_bytes_per_decode_step": mo["asked_bytes_per_decode_step"],
                                        "touched_bytes_per_decode_step": touched,
                                        "asked_over_touched": mo["asked_bytes_per_decode_step"] / max(1.0, touched),
                                        "tensor_level_hints_speedup": uvm["managed_hints"]["decode_tok_s"] / mo["decode_tok_s"],
                                        "explicit_ring_speedup": mo.get("explicit_ring_speedup_decode")}
    else:
        del r
        s.close()
        torch.cuda.empty_cache()
    if not args.no_configs and world == 1:
        # the other configurations, one pass each in a process of its own; this process gives its host pool and device memory back first
        del pool_np, pool
        if aliased:
            aliased.close()
        import gc
        gc.collect()
        torch.cuda.empty_cache()
        try:
            torch._C._host_emptyCache()
        except Exception:
            pass
        out["configs"] = other_config_summaries(args, max(120.0, 840.0 - (time.monotonic() - t_start)))
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def uvm_runs(args, cfg, lay, dev, pool, r, s, step_ms, T, only_demand):
    """The managed-memory runs of the same kernels under a ballast cap; reported, never fatal.  Frees the explicit
    engine's runner and session first (the ballast is sized from the free device memory)."""
    import torch
    from paper_2609_06172_b200 import binding as tb
    try:
        from paper_2609_06172_b200 import uvm_baseline
        s.close()
        r.arena = r.workspace = None
        torch.cuda.empty_cache()
        variants = (tb.VAR_MANAGED_DEMAND,) if only_demand else (tb.VAR_MANAGED_DEMAND, tb.VAR_MANAGED_HINTS, tb.VAR_MANAGED_OBJECT)
        uvm = uvm_baseline.run(cfg, lay, MACHINE, dev, lambda l, arr: arr.__setitem__(slice(None), pool.numpy()), variants=variants,
                               decode_cap=16 if lay.pool_bytes < (4 << 30) else 4, object_bytes=20 << 20)
        dec = cfg.B * T / (sum(step_ms[1:]) * 1e-3) if T else None
        for v in uvm.values():
            if dec and v.get("decode_tok_s"):
                v["explicit_ring_speedup_decode"] = dec / v["decode_tok_s"]
        return uvm
    except Exception as ex:
        return f"not run: {type(ex).__name__}: {ex}"


if __name__ == "__main__":
    main()
