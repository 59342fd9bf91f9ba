"""Managed-memory runs of the same kernels: the demand-paged baseline (no hints) and the hinted variant
(cudaMemPrefetchAsync for link-bound ops, cudaMemAdvise for the pin set), with the device capacity cut to
the budget by a ballast allocation, as the paper does with a helper process (Section V-A)."""
from __future__ import annotations

import ctypes

import numpy as np
import torch

from . import binding as tb
from .runner import Runner
from .session import Session


class ManagedPool:
    def __init__(self, nbytes):
        self.nbytes = nbytes
        self.ptr = tb.managed_alloc(nbytes)

    def numpy(self):
        return np.ctypeslib.as_array((ctypes.c_uint8 * self.nbytes).from_address(self.ptr))

    def free(self):
        if self.ptr:
            tb.managed_free(self.ptr)
            self.ptr = 0


def run(cfg, lay, machine, dev, fill, variants=(tb.VAR_MANAGED_DEMAND, tb.VAR_MANAGED_HINTS), decode_cap=16, slack=64 << 20, ballast=True,
        object_bytes=20 << 20):
    """Returns {variant name: {...}}.  `fill(layout, uint8 array)` writes the pool contents.  Capacity: the workspace
    and then a ballast tensor are allocated ONCE, before the GPU has touched the managed pool, so that budget + slack
    bytes of device memory are all the managed pages can ever occupy; both variants then run under that same cap
    (the driver caches chunks it evicted, so a cap computed after a managed run would be too generous).
    Decode is capped at `decode_cap` steps (demand paging under 2x oversubscription is slow); rates are per step."""
    torch.cuda.set_device(dev)
    out = {}
    pool = ManagedPool(lay.pool_bytes)
    try:
        fill(lay, pool.numpy())
        T = min(cfg.T, decode_cap)
        prompt = np.ascontiguousarray(_prompt(cfg))
        s = Session(lay, machine, pool_base=pool.ptr, pool_flags=tb.POOL_MANAGED)
        s.plan(T=T, variant=variants[0])
        r = Runner(s, cfg.B * cfg.S, device=str(dev), arena=False)
        hold, cap = None, {}
        if ballast:
            torch.cuda.synchronize()
            free, total = torch.cuda.mem_get_info(dev)
            nb = free - lay.budget - slack
            if nb > 0:
                try:
                    hold = torch.empty(nb, dtype=torch.uint8, device=dev)
                    cap["ballast_bytes"] = int(nb)
                except RuntimeError as ex:
                    cap["ballast"] = f"not allocated: {ex}"
            cap["device_bytes_left_for_managed_pages"] = int(torch.cuda.mem_get_info(dev)[0])
        for var in variants:
            name = {tb.VAR_MANAGED_DEMAND: "managed_demand", tb.VAR_MANAGED_HINTS: "managed_hints", tb.VAR_MANAGED_OBJECT: "managed_object"}[var]
            s.plan(T=T, variant=var)
            if var == tb.VAR_MANAGED_OBJECT:
                s.ctx.set_object_bytes(object_bytes)
            info = {"decode_steps": T, **cap}
            times = []
            for rep in range(2):                          # first pass warms code paths; second is reported
                tb.managed_evict(pool.ptr, lay.pool_bytes)
                r.reset()
                st = [r.step(tb.PREFILL, prompt, cfg.S, want_stats=True)]
                for _ in range(T):
                    st.append(r.step(tb.DECODE, None, 1, want_stats=True))
                times = [x.step_ms for x in st]
                asked = [int(x.h2d_bytes) for x in st]
            r.sync()
            info.update({"prefill_ms": times[0], "decode_ms_per_step": float(np.mean(times[1:])) if T else None,
                         "decode_tok_s": cfg.B * T / (sum(times[1:]) * 1e-3) if T else None,
                         "prefill_tok_s": cfg.B * cfg.S / (times[0] * 1e-3)})
            if var == tb.VAR_MANAGED_OBJECT:                  # bytes the object-level prefetcher asked for (resident or not)
                info.update({"object_bytes": int(object_bytes), "asked_bytes_prefill": asked[0],
                             "asked_bytes_per_decode_step": float(np.mean(asked[1:])) if T else None})
            out[name] = info
        del hold
        s.close()
        del r
        torch.cuda.empty_cache()
    finally:
        torch.cuda.synchronize()
        pool.free()
    return out


def _prompt(cfg):
    import seeded_inputs as si
    return si.prompt_tokens(cfg)
