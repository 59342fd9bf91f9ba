"""Oracle prefetch policy "P0": roofline classification, residency (pin) selection and the
ordered staging schedule.  Pure Python integers; no floating point anywhere.

TEST INFRASTRUCTURE - see oracle/__init__.py.

The paper describes the policy in prose only.  What it fixes, and where:
* three kernel classes - CGI(link)-bound, GPU-memory-bound, compute-bound - from a roofline
  with a compute roof, an HBM roof and a much lower CPU-GPU interconnect roof
  (Section III-C; Section IV-D "UVM Analyzer");
* prefetch exactly the tensors the upcoming kernel accesses, nothing else of the pool
  (Section IV-B, IV-E "Prefetch Engine");
* link-bound kernels trigger proactive prefetch; tensors reused across consecutive kernels
  are held resident during their reuse window (Section IV-D look-ahead affinity, IV-E).
Everything numeric below is this build's reading: the exact inequality, ties, the hold
window W_AFF, the zero-copy ratio ZC_DEN, the ring minimum, the 512-byte alignment.

Steps, in order (notation: P = peak flop/s, Bh = HBM bytes/s, Bl = host-link bytes/s):

1. classify each op i with mig_i = sum of touched bytes of its pool accesses:
     LINK    iff mig_i*P > flops_i*Bl and mig_i*Bh > hbm_i*Bl   (the link time exceeds both others)
     COMPUTE iff not LINK and flops_i*Bh >= hbm_i*P
     HBM     otherwise.                With the P bit off every op with mig_i > 0 is LINK.
2. crit[t] iff a LINK op accesses t;  score[t] = link bytes residency would save: over LINK-op accesses,
   the touched bytes, plus the tensor's size for each write (a written stay ends in a whole-tensor D2H).
3. zero-copy (ZC bit): a READONLY tensor whose every access touches < size/ZC_DEN bytes is read
   in place over the link and never staged.
4. residency episodes: consecutive accesses of t (same step, gap <= W_AFF ops) share one stay.
   live_i = aligned bytes of all non-ZC episodes covering op i; ring_min = 2 * max_i live_i;
   error if ring_min > budget.  pin_cap = budget - ring_min.
5. pins (A bit): candidates score > 0, non-ZC, by density score/size descending (exact cross
   products), tie -> lower id.  Groups of equal density are taken in turn: a group that fits is
   pinned whole; one that does not has its share of pinned bytes spread evenly along the id order
   by integer error diffusion (err += a*cap; pin iff err >= a*total; then err -= a*total), followed
   by a greedy fill with skip.  Spreading keeps the link demand of the streamed rest uniform over a
   step instead of leaving the copy engine idle while compute walks a pinned prefix of layers.
   Pins sit at [0, used) in the order they were chosen; the ring is [used, budget).
5b. windowed reservation (W bit): a pinned tensor that is born on the device (MUTABLE, first access a write, no data
   in the pool) in step s >= 2 - a KV tile of positions not yet reached - does not need its slot before that step.
   Adjacent such slots with the same birth step form a vacancy region, free for steps [0, s).  Regions are taken by
   longest vacancy first (tie: lower offset); the unpinned, non-ZC, READONLY candidates of step 5, in the same density
   order, become tenants by first fit: a tenant accessed in at least two steps before s is loaded at its first access
   into the region (bump allocation) and stays there until its last access before step s, after which it is streamed
   through the ring like any unpinned tensor.  The landlord's own placement waits for the last use of every tenant
   of its region.  Saves the tenant's size once per step of the vacancy but the first.
6. schedule: walk ops in order, accesses in list order.
     pinned tensor, first access: LOAD (H2D into its slot), or ALLOC if MUTABLE and the access is W.
     ring tensor, episode start: FIFO bump allocation (wrap to the ring base when the tail does
       not fit), evicting the oldest stays it overlaps; wait_op = running max of the evicted stays'
       last-use ops (and, for a MUTABLE tensor, of the op after which it was last written back);
       kind H2D, or ALLOC when MUTABLE, never written and the access is W.
       wait_op >= first_use -> error (ring too small).
     ring tensor, episode end, written during the stay: D2H of the whole tensor after that op.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass
from typing import Dict, List, Tuple

ALIGN = 512
W_AFF = 4
ZC_DEN = 2
CLS_LINK, CLS_HBM, CLS_COMPUTE = 0, 1, 2
CMD_H2D, CMD_ALLOC, CMD_D2H = 0, 1, 2
BIT_A, BIT_P, BIT_ZC, BIT_W = 1, 2, 4, 8
MODE_R, MODE_W = 1, 2
F_READONLY, F_MUTABLE = 1, 2


class PlanError(Exception):
    pass


@dataclass
class Machine:
    peak_flops: int
    hbm_Bps: int
    h2d_Bps: int
    d2h_Bps: int


@dataclass
class Cmd:
    seq: int
    kind: int
    tensor: int
    nbytes: int
    pool_off: int
    arena_off: int
    wait_op: int
    first_use: int
    release_after: int

    def pack(self) -> bytes:
        return struct.pack("<IBIQQQiii", self.seq, self.kind, self.tensor, self.nbytes, self.pool_off,
                           self.arena_off, self.wait_op, self.first_use, self.release_after)


def alignup(x: int) -> int:
    return (x + ALIGN - 1) // ALIGN * ALIGN


def classify(flops: int, hbm: int, mig: int, m: Machine, bit_p: bool = True, measured_ns: int = 0) -> int:
    """measured_ns > 0: the runtime monitor's kernel time replaces both analytic roofs in the link test
    (Section IV-E "Runtime Monitor": classes are re-evaluated from measured kernel time): LINK iff moving the op's
    pool bytes over the link takes longer than the kernel itself ran, mig / Bl > t  <=>  mig * 1e9 > t_ns * Bl."""
    if mig > 0 and not bit_p:
        return CLS_LINK
    if measured_ns > 0:
        if mig * 1_000_000_000 > measured_ns * m.h2d_Bps:
            return CLS_LINK
        return CLS_COMPUTE if flops * m.hbm_Bps >= hbm * m.peak_flops else CLS_HBM
    if mig * m.peak_flops > flops * m.h2d_Bps and mig * m.hbm_Bps > hbm * m.h2d_Bps:
        return CLS_LINK
    if flops * m.hbm_Bps >= hbm * m.peak_flops:
        return CLS_COMPUTE
    return CLS_HBM


@dataclass
class Plan:
    cls: List[int]
    crit: List[int]
    score: List[int]
    zc: List[int]
    pins: List[Tuple[int, int]]
    ring_base: int
    ring_size: int
    cmds: List[Cmd]
    totals: List[Tuple[int, int, int, int]]       # per step (h2d bytes, d2h bytes, zc bytes, n cmds)
    episodes: List[Tuple[int, int, int]]          # (tensor, first op, last op) of ring stays (diagnostic)

    def blobs(self) -> Dict[str, bytes]:
        return {
            "classes": bytes(self.cls),
            "tensors": b"".join(struct.pack("<BBQ", self.crit[t], self.zc[t], self.score[t]) for t in range(len(self.crit))),
            "pins": b"".join(struct.pack("<IQ", t, o) for t, o in self.pins) + struct.pack("<QQ", self.ring_base, self.ring_size),
            "commands": b"".join(c.pack() for c in self.cmds),
            "totals": b"".join(struct.pack("<QQQQ", *x) for x in self.totals),
        }


def plan(tensors, ops, steps, machine: Machine, budget: int, bits: int = BIT_A | BIT_P | BIT_ZC | BIT_W, measured_ns=None,
         written_before=(), resident=None) -> Plan:
    """tensors: list of objects with .size .pool_off .flags; ops: list with .step .flops .hbm .acc;
    steps: [(kind, first op, count)]; measured_ns: optional per-op kernel times in integer nanoseconds (0 = none);
    written_before: tensors that already hold data in the pool when the trace starts (a tail re-plan), whose first
    access therefore loads them even if it is a write."""
    T, N = len(tensors), len(ops)
    # 1-2: classes, criticality, score
    cls = []
    crit = [0] * T
    score = [0] * T
    for i, op in enumerate(ops):
        mig = sum(a[2] for a in op.acc)
        c = classify(op.flops, op.hbm, mig, machine, bool(bits & BIT_P), int(measured_ns[i]) if measured_ns is not None else 0)
        cls.append(c)
        if c == CLS_LINK:
            for (t, mode, touched) in op.acc:
                crit[t] = 1
                score[t] += touched + (tensors[t].size if mode & MODE_W else 0)
    # 3: zero-copy
    accessed = [0] * T
    sparse = [1] * T
    for op in ops:
        for (t, _, touched) in op.acc:
            accessed[t] = 1
            if touched * ZC_DEN >= tensors[t].size:
                sparse[t] = 0
    zc = [1 if (bits & BIT_ZC) and accessed[t] and sparse[t] and tensors[t].flags == F_READONLY else 0 for t in range(T)]
    # 4: episodes from the trace alone
    step_of = [op.step for op in ops]
    acc_ops: Dict[int, List[int]] = {}
    for i, op in enumerate(ops):
        for (t, _, _) in op.acc:
            if not zc[t]:
                lst = acc_ops.setdefault(t, [])
                if not lst or lst[-1] != i:
                    lst.append(i)
    episodes_of: Dict[int, List[Tuple[int, int]]] = {}
    for t, lst in acc_ops.items():
        eps = []
        first = last = lst[0]
        for i in lst[1:]:
            if i <= last + W_AFF and step_of[i] == step_of[last]:
                last = i
            else:
                eps.append((first, last))
                first = last = i
        eps.append((first, last))
        episodes_of[t] = eps
    delta = [0] * (N + 1)
    for t, eps in episodes_of.items():
        a = alignup(tensors[t].size)
        for (f, l) in eps:
            delta[f] += a
            delta[l + 1] -= a
    wmax = live = 0
    for i in range(N):
        live += delta[i]
        wmax = max(wmax, live)
    ring_min = 2 * wmax
    if ring_min > budget:
        raise PlanError("budget smaller than the ring minimum")
    pin_cap = budget - ring_min
    # 5: pins
    pinned_off: Dict[int, int] = {}
    used = 0
    if bits & BIT_A:
        cands = [t for t in range(T) if score[t] > 0 and not zc[t]]
        import functools

        def cmp(a, b):
            lhs, rhs = score[a] * tensors[b].size, score[b] * tensors[a].size
            if lhs != rhs:
                return -1 if lhs > rhs else 1
            return -1 if a < b else (1 if a > b else 0)

        order = sorted(cands, key=functools.cmp_to_key(cmp))
        g0 = 0
        while g0 < len(order):
            # group of equal density (exact cross products against the group's first tensor)
            g1 = g0 + 1
            while g1 < len(order) and score[order[g1]] * tensors[order[g0]].size == score[order[g0]] * tensors[order[g1]].size:
                g1 += 1
            group = order[g0:g1]
            g0 = g1
            cap_left = pin_cap - used
            total = sum(alignup(tensors[t].size) for t in group)
            if total > cap_left:
                # not all fit: spread the pinned bytes evenly along the id (= first-use) order by error
                # diffusion, so that the link demand of the rest is uniform over a step
                err = 0
                for t in group:
                    a = alignup(tensors[t].size)
                    err += a * cap_left
                    if err >= a * total:
                        err -= a * total
                        pinned_off[t] = used
                        used += a
            for t in group:                                   # everything that fits / greedy fill, with skip
                a = alignup(tensors[t].size)
                if t not in pinned_off and used + a <= pin_cap:
                    pinned_off[t] = used
                    used += a
    # 5a: pins that are resident already (a plan made in the middle of a run, see plan_tail): a chosen tensor that is on the
    # device keeps its place and is not loaded again; the others go, in the order they were chosen, into the first gap
    # between the kept ones that holds them (none: not pinned after all).  The pin region ends where the longer of the
    # two layouts ends.
    kept: Dict[int, int] = {}
    if resident is not None:
        kept = {t: resident[t] for t in pinned_off if t in resident}
        chosen = sorted(pinned_off, key=pinned_off.get)
        region_end = max([used] + [o + alignup(tensors[t].size) for t, o in kept.items()])
        holes, pos = [], 0
        for (a0, a1) in sorted((o, o + alignup(tensors[t].size)) for t, o in kept.items()):
            if a0 > pos:
                holes.append([pos, a0])
            pos = max(pos, a1)
        if pos < region_end:
            holes.append([pos, region_end])
        placed = dict(kept)
        for t in chosen:
            if t in kept:
                continue
            a = alignup(tensors[t].size)
            for h in holes:
                if h[1] - h[0] >= a:
                    placed[t] = h[0]
                    h[0] += a
                    break
        pinned_off, used = placed, region_end
        if budget - used < ring_min:
            raise PlanError("kept pins leave less than the ring minimum")
    ring_base, ring_size = used, budget - used
    pins = sorted(pinned_off.items())
    # 5b: windowed reservation - tenants of the slots of pinned tensors that are born late (not in a plan that keeps pins)
    tenancy: Dict[int, Tuple[int, int]] = {}       # tenant -> (arena offset, last op it is used there)
    landlord_wait: Dict[int, int] = {}             # late-born pinned tensor -> op its placement must wait for
    if (bits & BIT_W) and pinned_off and resident is None:
        first_acc: Dict[int, Tuple[int, int]] = {}
        for i, op in enumerate(ops):
            for (t, mode, _) in op.acc:
                first_acc.setdefault(t, (i, mode))
        late = [t for t in pinned_off if tensors[t].flags == F_MUTABLE and t not in written_before
                and first_acc[t][1] == MODE_W and step_of[first_acc[t][0]] >= 2]
        regions = []                               # [start, end, birth step, landlords]
        for t in sorted(late, key=lambda t: pinned_off[t]):
            o, a, b = pinned_off[t], alignup(tensors[t].size), step_of[first_acc[t][0]]
            if regions and regions[-1][1] == o and regions[-1][2] == b:
                regions[-1][1] = o + a
                regions[-1][3].append(t)
            else:
                regions.append([o, o + a, b, [t]])
        regions.sort(key=lambda r: (-r[2], r[0]))
        fill = [r[0] for r in regions]
        region_wait = [-1] * len(regions)
        for t in order:
            if t in pinned_off or tensors[t].flags != F_READONLY:
                continue
            a = alignup(tensors[t].size)
            for k, (start, end, b, _) in enumerate(regions):
                if fill[k] + a > end:
                    continue
                before = [i for i in acc_ops[t] if step_of[i] < b]
                if not before or step_of[before[0]] == step_of[before[-1]]:
                    continue                       # used in fewer than two steps of the vacancy: nothing to save
                tenancy[t] = (fill[k], before[-1])
                fill[k] += a
                region_wait[k] = max(region_wait[k], before[-1])
                break
        for k, r in enumerate(regions):
            for t in r[3]:
                landlord_wait[t] = region_wait[k]
    # 6: schedule
    cmds: List[Cmd] = []
    totals = [[0, 0, 0, 0] for _ in steps]
    ep_index = {t: 0 for t in episodes_of}
    open_stay: Dict[int, int] = {}            # ring tensor -> arena offset of its current stay
    pin_loaded = set(kept)
    written_ever = set(written_before)
    last_wb_op: Dict[int, int] = {}
    fifo: List[Tuple[int, int, int]] = []     # (start, end, last-use op) of ring stays, oldest first
    head = 0
    run_wait = -1
    ending: Dict[int, List[int]] = {}         # op -> ring tensors whose stay ends there
    dirty_now = set()
    ep_list = []

    def emit(kind, t, arena_off, wait, first, release):
        c = Cmd(len(cmds), kind, t, tensors[t].size, tensors[t].pool_off, arena_off, wait, first, release)
        cmds.append(c)
        tot = totals[step_of[first]]
        tot[3] += 1
        if kind == CMD_H2D:
            tot[0] += c.nbytes
        elif kind == CMD_D2H:
            tot[1] += c.nbytes

    for i, op in enumerate(ops):
        for (t, mode, touched) in op.acc:
            if zc[t]:
                totals[op.step][2] += touched
                continue
            mutable = tensors[t].flags == F_MUTABLE
            fresh_write = mutable and mode == MODE_W and t not in written_ever
            if t in pinned_off:
                if t not in pin_loaded:
                    pin_loaded.add(t)
                    emit(CMD_ALLOC if fresh_write else CMD_H2D, t, pinned_off[t], landlord_wait.get(t, -1), i, N - 1)
            elif t in tenancy and i <= tenancy[t][1]:
                if t not in pin_loaded:                        # a tenant: loaded once into the vacant slot, used there
                    pin_loaded.add(t)
                    emit(CMD_H2D, t, tenancy[t][0], -1, i, tenancy[t][1])
            elif t not in open_stay:
                while episodes_of[t][ep_index[t]][0] < i:      # stays a tenancy made unnecessary
                    ep_index[t] += 1
                f, l = episodes_of[t][ep_index[t]]
                assert f == i
                a = alignup(tensors[t].size)
                if a > ring_size:
                    raise PlanError("tensor larger than the ring")
                evicted = -1
                if head + a > ring_size:                       # tail does not fit: skip it, wrap
                    while fifo and fifo[0][0] >= head:
                        evicted = max(evicted, fifo.pop(0)[2])
                    head = 0
                while fifo and fifo[0][0] < head + a and fifo[0][1] > head:
                    evicted = max(evicted, fifo.pop(0)[2])
                run_wait = max(run_wait, evicted, last_wb_op.get(t, -1))
                if run_wait >= i:
                    raise PlanError("ring too small: a stay would wait on its own op")
                fifo.append((head, head + a, l))
                open_stay[t] = ring_base + head
                emit(CMD_ALLOC if fresh_write else CMD_H2D, t, ring_base + head, run_wait, i, l)
                ending.setdefault(l, []).append(t)
                ep_list.append((t, f, l))
                head += a
            if mode & MODE_W:
                written_ever.add(t)
                if t not in pinned_off:
                    dirty_now.add(t)
        for t in ending.pop(i, []):                            # stays that end at this op
            off = open_stay.pop(t)
            if t in dirty_now:
                dirty_now.discard(t)
                emit(CMD_D2H, t, off, i, i, i)
                last_wb_op[t] = i
            ep_index[t] += 1
    return Plan(cls, crit, score, zc, pins, ring_base, ring_size, cmds, [tuple(x) for x in totals], ep_list)


def plan_tail(tensors, ops, steps, machine: Machine, budget: int, first_step: int, bits: int = BIT_A | BIT_P | BIT_ZC | BIT_W,
              measured_ns=None, resident=None) -> Plan:
    """Re-plan at a step boundary, while the run is under way (Section IV-E "Runtime Monitor": classes are re-evaluated
    from measured kernel times and the engine adapts; the paper does not say how the switch is made).  Reading: the
    steps from first_step on are planned as a trace of their own, with the same policy.  At the boundary the engine has
    drained - every stay has ended (stays never cross a step) and every written pinned tensor has been written back -
    so nothing is resident and the pool is up to date: the tail plan starts from an empty arena, and a tensor written in
    an earlier step holds data, so its first access loads it (H2D) even when that access is a write.
    measured_ns: one entry per op of the WHOLE trace (0 = not measured).  Op indices in the returned commands are those
    of the whole trace; classes and per-step totals cover the tail only.
    resident (tensor -> arena offset): the pinned tensors of the plan in use that are on the device at the boundary.  Given,
    the switch keeps them: those the tail plan pins again stay where they are, hold the newest data (the engine then
    writes back only the written pins it gives up) and are not loaded again; the windowed reservation is not applied."""
    import copy
    first_op = steps[first_step][1]
    written = set()
    for op in ops[:first_op]:
        for (t, mode, _) in op.acc:
            if mode & MODE_W:
                written.add(t)
    sub_ops = []
    for op in ops[first_op:]:
        o = copy.copy(op)
        o.step = op.step - first_step
        sub_ops.append(o)
    sub_steps = [(k, o0 - first_op, n) for (k, o0, n) in steps[first_step:]]
    pl = plan(tensors, sub_ops, sub_steps, machine, budget, bits,
              None if measured_ns is None else list(measured_ns[first_op:]), written_before=written, resident=resident)
    for c in pl.cmds:
        if c.wait_op >= 0:
            c.wait_op += first_op
        c.first_use += first_op
        c.release_after += first_op
    pl.episodes = [(t, f + first_op, l + first_op) for (t, f, l) in pl.episodes]
    return pl
