"""Independent validator for a prefetch plan (from the oracle or from the library).

TEST INFRASTRUCTURE - see oracle/__init__.py.

It knows nothing of how a plan was made.  It parses the canonical blobs, replays the
commands against a versioned model of host pool and device arena, and checks the
properties any correct schedule for the paper's problem must have (Section IV-E: the
tensors a kernel needs are on the device before it runs, inside a fixed capacity):

 I1 resident at use : every (op, tensor) access finds that tensor's bytes in the arena
                      (a stay with first_use <= op <= release_after whose copy could start
                      before the op: wait_op < first_use), or the tensor is zero-copy.
 I2 budget          : every placement lies in [0, budget); a placement never overlaps a stay
                      still needed (its release_after must be <= the placement's wait_op);
                      pins do not overlap the ring or each other.  A tensor that is not pinned may be
                      placed inside the pin region only as a tenant: wholly inside slots of pinned
                      tensors that have not been placed yet, disjoint from live tenants, and every
                      pin placement waits for the last use of the tenants of its slot.
 I3 cover           : each (tensor, first_use) appears exactly once; placements are ordered by
                      (first_use, position in that op's access list); a write-back follows the
                      placements of its op and precedes those of the next op.
 I4 no self-wait    : wait_op < first_use, and wait_op is non-decreasing over ring placements.
 I5 write-back      : with version counters per tensor, every read sees the newest version and
                      every copy from the host copies the newest version.
"""
from __future__ import annotations

import struct

CMD_H2D, CMD_ALLOC, CMD_D2H = 0, 1, 2
ALIGN = 512


class PlanInvalid(Exception):
    pass


def parse(blobs, n_tensors):
    cmds = []
    raw = blobs["commands"]
    rec = struct.Struct("<IBIQQQiii")
    for k in range(0, len(raw), rec.size):
        cmds.append(rec.unpack_from(raw, k))
    tb = blobs["tensors"]
    crit, zc, score = [], [], []
    for t in range(n_tensors):
        c, z, s = struct.unpack_from("<BBQ", tb, t * 10)
        crit.append(c), zc.append(z), score.append(s)
    pb = blobs["pins"]
    npin = (len(pb) - 16) // 12
    pins = [struct.unpack_from("<IQ", pb, 12 * k) for k in range(npin)]
    ring_base, ring_size = struct.unpack_from("<QQ", pb, 12 * npin)
    tot = blobs["totals"]
    totals = [struct.unpack_from("<QQQQ", tot, k) for k in range(0, len(tot), 32)]
    return dict(cmds=cmds, crit=crit, zc=zc, score=score, pins=pins, ring_base=ring_base,
                ring_size=ring_size, totals=totals, classes=list(blobs["classes"]))


def check(tensors, ops, steps, budget, blobs, first_step=0, resident=None):
    """Raises PlanInvalid with a reason; returns a small summary dict when everything holds.
    first_step > 0: `blobs` is a tail plan made at that step boundary for the rest of the trace (op indices of the
    whole trace); the replay then starts from an empty arena with every tensor written in an earlier step holding
    data in the pool, so such a tensor may never be placed by ALLOC.
    resident (tensor -> arena offset): pinned tensors that are on the device at the boundary, with the newest data; a pin
    of the tail plan at the same offset starts the replay resident (the pool's copy of one written earlier is stale: it
    was not written back), and must not be placed again."""
    P = parse(blobs, len(tensors))
    first_op = steps[first_step][1]
    written_before = {t for op in ops[:first_op] for (t, mode, _) in op.acc if mode & 2}
    if first_step:
        import copy
        tail = []
        for op in ops[first_op:]:
            o = copy.copy(op)
            o.step = op.step - first_step
            tail.append(o)
        ops, steps = tail, [(k, o0 - first_op, n) for (k, o0, n) in steps[first_step:]]
        P["cmds"] = [(q, kind, t, nb, po, ao, (w - first_op if w >= 0 else w), f - first_op, r - first_op)
                     for (q, kind, t, nb, po, ao, w, f, r) in P["cmds"]]
        if any(c[6] < -1 or c[7] < 0 for c in P["cmds"]):
            raise PlanInvalid("a tail command refers to an op before the boundary")
    N = len(ops)
    if len(P["classes"]) != N:
        raise PlanInvalid("class count")
    up = lambda x: (x + ALIGN - 1) // ALIGN * ALIGN
    # pins: disjoint, before the ring
    pin_off = dict(P["pins"])
    spans = sorted((o, o + up(tensors[t].size)) for t, o in P["pins"])
    for (a, b), (c, d) in zip(spans, spans[1:]):
        if b > c:
            raise PlanInvalid("pins overlap")
    if spans and spans[-1][1] > P["ring_base"]:
        raise PlanInvalid("pin region runs into the ring")
    if P["ring_base"] + P["ring_size"] != budget:
        raise PlanInvalid("ring does not end at the budget")
    # group commands by first_use
    by_op = {}
    seen = set()
    last_first = -1
    for c in P["cmds"]:
        seq, kind, t, nbytes, pool_off, arena_off, wait, first, rel = c
        if first < last_first:
            raise PlanInvalid("commands not ordered by first use")
        last_first = first
        if nbytes != tensors[t].size or pool_off != tensors[t].pool_off:
            raise PlanInvalid("command does not name the tensor's pool range")
        if arena_off % ALIGN or arena_off + nbytes > budget:
            raise PlanInvalid("placement outside the budget or unaligned")
        if kind != CMD_D2H:
            if (t, first) in seen:
                raise PlanInvalid("tensor placed twice for one op")
            seen.add((t, first))
            if not (wait < first <= rel):
                raise PlanInvalid("self-wait or empty stay")
        by_op.setdefault(first, []).append(c)
    for k, c in enumerate(P["cmds"]):
        if c[0] != k:
            raise PlanInvalid("sequence numbers")
    # replay
    host_ver = [1 if t in written_before else 0 for t in range(len(tensors))]
    newest = list(host_ver)
    stays = {}                      # tensor -> [arena_off, release_after, version held, is_pin]
    for t, off in (resident or {}).items():
        if pin_off.get(t) == off:
            stays[t] = [off, N - 1, newest[t], True]
            if newest[t]:
                host_ver[t] = 0     # written on the device, not written back at the switch
    placed = []                     # (start, end, release_after) of ring stays not yet overwritten
    tenants = []                    # (start, end, release_after) of placements of unpinned tensors inside the pin region
    ring_wait = -1
    h2d = [0] * len(steps)
    d2h = [0] * len(steps)
    zcb = [0] * len(steps)
    ncmd = [0] * len(steps)
    pending_wb = {}                 # tensor -> op of last write-back
    ends_at = {}                    # op -> ring tensors whose stay ends there
    for i, op in enumerate(ops):
        cl = by_op.get(i, [])
        places = [c for c in cl if c[1] != CMD_D2H]
        wbs = [c for c in cl if c[1] == CMD_D2H]
        if cl and [c[1] == CMD_D2H for c in cl] != [False] * len(places) + [True] * len(wbs):
            raise PlanInvalid("write-backs must follow the op's placements")
        # placements must follow the order of the op's access list
        order = [a[0] for a in op.acc]
        idx = [order.index(c[2]) if c[2] in order else -1 for c in places]
        if -1 in idx or idx != sorted(idx):
            raise PlanInvalid("placements not in access-list order")
        for c in places:
            seq, kind, t, nbytes, pool_off, arena_off, wait, first, rel = c
            is_pin = t in pin_off
            if is_pin:
                if arena_off != pin_off[t] or t in stays:
                    raise PlanInvalid("pin loaded twice or at the wrong slot")
                s, e = arena_off, arena_off + up(nbytes)
                for (a, b, r) in tenants:
                    if a < e and b > s and r > wait:
                        raise PlanInvalid(f"pin placed over a tenant still needed until op {r}")
            elif arena_off < P["ring_base"]:
                # a tenant of slots whose pinned tensors are not there yet
                s, e = arena_off, arena_off + up(nbytes)
                if e > P["ring_base"] or kind != CMD_H2D:
                    raise PlanInvalid("tenant placement leaves the pin region or is not a load")
                covered = 0
                for (pt, po) in P["pins"]:
                    a, b = po, po + up(tensors[pt].size)
                    if a < e and b > s:
                        if pt in stays:
                            raise PlanInvalid("tenant placed over a pinned tensor that is resident")
                        covered += min(b, e) - max(a, s)
                if covered != e - s:
                    raise PlanInvalid("tenant placement not wholly inside pin slots")
                for (a, b, r) in tenants:
                    if a < e and b > s and r >= first:
                        raise PlanInvalid("two tenants overlap in place and time")
                tenants.append((s, e, rel))
                if t in stays and stays[t][1] >= first:
                    raise PlanInvalid("tensor has two overlapping stays")
            else:
                if wait < ring_wait:
                    raise PlanInvalid("ring waits must be non-decreasing")
                ring_wait = wait
                s, e = arena_off, arena_off + up(nbytes)
                keep = []
                for (a, b, r) in placed:
                    if a < e and b > s:
                        if r > wait:
                            raise PlanInvalid(f"placement for op {first} overwrites a stay needed until op {r}")
                    else:
                        keep.append((a, b, r))
                placed = keep + [(s, e, rel)]
                if t in stays and stays[t][1] >= first:
                    raise PlanInvalid("tensor has two overlapping stays")
                if t in pending_wb and wait < pending_wb[t]:
                    raise PlanInvalid("reload may start before the previous write-back")
            if kind == CMD_H2D:
                if host_ver[t] != newest[t]:
                    raise PlanInvalid(f"H2D of tensor {t} copies a stale host version")
                ver = host_ver[t]
                h2d[op.step] += nbytes
            else:
                ver = None if newest[t] else 0
                if newest[t]:
                    raise PlanInvalid("ALLOC of a tensor that already holds data")
            stays[t] = [arena_off, rel, ver, is_pin]
            if not is_pin:
                ends_at.setdefault(rel, []).append(t)
            ncmd[op.step] += 1
        for (t, mode, touched) in op.acc:
            if P["zc"][t]:
                if mode & 2:
                    raise PlanInvalid("write through a zero-copy tensor")
                zcb[op.step] += touched
                continue
            st = stays.get(t)
            if st is None or not (i <= st[1]):
                raise PlanInvalid(f"op {i} accesses tensor {t} that is not resident")
            if mode & 1 and st[2] != newest[t]:
                raise PlanInvalid(f"op {i} reads a stale copy of tensor {t}")
            if mode & 2:
                newest[t] += 1
                st[2] = newest[t]
        for c in wbs:
            seq, kind, t, nbytes, pool_off, arena_off, wait, first, rel = c
            st = stays.get(t)
            if st is None or st[0] != arena_off or st[1] != i or wait != i:
                raise PlanInvalid("write-back does not match a stay ending at this op")
            host_ver[t] = st[2]
            pending_wb[t] = i
            d2h[op.step] += nbytes
            ncmd[op.step] += 1
        # stays that end here and were written but not written back lose data
        for t in ends_at.pop(i, []):
            if stays[t][2] != host_ver[t]:
                raise PlanInvalid(f"stay of tensor {t} ends dirty without a write-back")
            del stays[t]
    got = [tuple(x) for x in zip(h2d, d2h, zcb, ncmd)]
    if got != [tuple(x) for x in P["totals"]]:
        raise PlanInvalid("per-step totals do not match the commands")
    return {"h2d": sum(h2d), "d2h": sum(d2h), "zc": sum(zcb), "n_cmds": len(P["cmds"]), "n_pins": len(pin_off)}
