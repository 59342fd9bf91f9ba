"""Device plumbing for a planned session: PyTorch supplies pinned host memory, device buffers and
streams; every computation happens inside libtgp.so."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as tb
from .session import Session


def pinned_pool(nbytes: int) -> torch.Tensor:
    """Page-locked host buffer for the pool (512-byte aligned by the CUDA host allocator)."""
    t = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    assert t.data_ptr() % 512 == 0
    return t


class AliasedPool:
    """Host pool for shapes whose weights exceed what this host can page-lock: the weight regions of layers l and
    l + phys_layers, l + 2 * phys_layers, ... are the same physical pages (one memfd mapped several times into one
    contiguous virtual range), so the pool keeps its full virtual layout - every tensor at its own address, nothing the
    library could tell apart - while physical memory holds only phys_layers layers.  Bytes moved over the link and
    arithmetic per step are unchanged; the weights of aliased layers are equal, so logits are those of another model:
    for throughput runs only.  Embedding, head and KV tiles are never aliased.  The memory is not page-locked yet:
    page_lock() registers it mapping by mapping (one cudaHostRegister over several mappings is refused by the OS layer),
    after which the pool is registered with POOL_PINNED."""

    def __init__(self, layout, phys_layers):
        import ctypes as C
        import mmap
        import os
        import seeded_inputs as si
        cfg = layout.cfg
        kv = (si.K_KT, si.K_VT)
        start = [min(t.pool_off for t in layout.tensors if t.layer == l and t.kind not in kv) for l in range(cfg.L)]
        end = max(t.pool_off + t.size for t in layout.tensors if t.layer == cfg.L - 1 and t.kind not in kv)
        lb = (end - start[0]) // cfg.L
        page = mmap.PAGESIZE
        if any(start[l] != start[0] + l * lb for l in range(cfg.L)) or end != start[0] + cfg.L * lb or lb % page or start[0] % page:
            raise ValueError("layer regions are not contiguous, equal and page-aligned")
        if not 1 <= phys_layers <= cfg.L:
            raise ValueError("phys_layers out of range")
        self.nbytes = layout.pool_bytes
        self.layer_bytes, self.first_layer_off, self.phys_layers = lb, start[0], phys_layers
        vlen = (self.nbytes + page - 1) // page * page
        tail_v = start[0] + cfg.L * lb                                  # first virtual byte after the layers
        self.phys_bytes = start[0] + phys_layers * lb + (vlen - tail_v)
        libc = C.CDLL(None, use_errno=True)
        libc.mmap.restype, libc.mmap.argtypes = C.c_void_p, [C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_int, C.c_long]
        libc.munmap.restype, libc.munmap.argtypes = C.c_int, [C.c_void_p, C.c_size_t]
        self._libc, self._vlen = libc, vlen
        self._fd = os.memfd_create("tgp_pool")
        os.ftruncate(self._fd, self.phys_bytes)
        failed = C.c_void_p(-1).value                                   # MAP_FAILED; protection 0 below is PROT_NONE: address space only
        base = libc.mmap(None, vlen, 0, mmap.MAP_PRIVATE | mmap.MAP_ANONYMOUS | getattr(mmap, "MAP_NORESERVE", 0x4000), -1, 0)
        if base in (None, failed):
            raise OSError(C.get_errno(), "mmap (reserve) failed")
        self._base = base

        self.pieces = []                                                # (virtual offset, length) of every mapping

        def place(voff, length, foff):
            got = libc.mmap(C.c_void_p(base + voff), length, mmap.PROT_READ | mmap.PROT_WRITE, mmap.MAP_SHARED | 0x10, self._fd, foff)   # 0x10 = MAP_FIXED
            if got != base + voff:
                raise OSError(C.get_errno(), "mmap (place) failed")
            self.pieces.append((voff, length))

        place(0, start[0], 0)                                           # embedding
        for l0 in range(0, cfg.L, phys_layers):                         # each group of layers onto the same file range
            n = min(phys_layers, cfg.L - l0)
            place(start[0] + l0 * lb, n * lb, start[0])
        place(tail_v, vlen - tail_v, start[0] + phys_layers * lb)        # final norm, head, KV tiles
        self._buf = (C.c_uint8 * self.nbytes).from_address(base)

    def data_ptr(self):
        return self._base

    def page_lock(self):
        """cudaHostRegister, one call per mapping.  Raises on the first refusal (what was registered stays registered
        until close())."""
        rt = torch.cuda.cudart()
        self._locked = getattr(self, "_locked", [])
        for voff, length in self.pieces:
            rc = int(rt.cudaHostRegister(self._base + voff, length, 0))
            if rc != 0:
                raise RuntimeError(f"cudaHostRegister refused {length} bytes at pool offset {voff}: cudaError {rc}")
            self._locked.append(voff)

    def numpy(self):
        return np.ctypeslib.as_array(self._buf)

    def close(self):
        import os
        if self._base:
            for voff in getattr(self, "_locked", []):
                torch.cuda.cudart().cudaHostUnregister(self._base + voff)
            self._locked = []
            self._buf = None
            self._libc.munmap(self._base, self._vlen)
            os.close(self._fd)
            self._base = 0


class Runner:
    """Owns arena, workspace, logits and streams for one Session and drives tgp_step()."""

    def __init__(self, session: Session, max_tokens: int, device="cuda:0", arena=True):
        self.s = session
        cfg = session.layout.cfg
        self.cfg = cfg
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.ws_bytes = tb.model_workspace_bytes(session.cfg, max_tokens)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.dev)
        self.arena_bytes = session.layout.budget
        self.arena = torch.empty((self.arena_bytes + 511) // 512 * 512, dtype=torch.uint8, device=self.dev) if arena else None
        assert (self.arena is None or self.arena.data_ptr() % 512 == 0) and self.workspace.data_ptr() % 256 == 0
        self.logits = torch.empty((cfg.B, cfg.V), dtype=torch.float32, device=self.dev)
        self.argmax = torch.empty((cfg.B,), dtype=torch.int32, device=self.dev)
        self.compute = torch.cuda.Stream(device=self.dev)
        self.copy = torch.cuda.Stream(device=self.dev)
        if arena:
            session.attach_device(self.arena, self.arena_bytes, self.workspace, self.ws_bytes, max_tokens)
        else:                                   # managed variants read the pool in place: no arena
            session.ctx.model_bind(session.cfg, session.roles, session.router_bias, self.workspace, self.ws_bytes, max_tokens)

    def reset(self):
        self.s.ctx.run_reset()

    def step(self, kind, tokens, q_len, want_stats=False):
        """tokens: int32 numpy / pinned tensor [B, q_len] on the host, or None to feed the last argmax."""
        return self.s.ctx.step(kind, tokens, self.cfg.B, q_len, self.logits, self.argmax, self.compute, self.copy, want_stats)

    def sync(self):
        self.compute.synchronize()
        self.copy.synchronize()
        torch.cuda.synchronize(self.dev)

    def generate(self, prompt: np.ndarray, n_decode: int, forced=None, keep_logits=True):
        """Prefill + n_decode steps.  forced [B, n_decode]: teacher-forced tokens; else the device argmax is fed
        back without leaving the GPU.  Returns (list of logits arrays per step, tokens [B, n_decode])."""
        self.reset()
        out, toks = [], []
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        self.step(tb.PREFILL, prompt, prompt.shape[1])
        for t in range(n_decode + 1):
            if keep_logits or t == n_decode:
                self.compute.synchronize()
                out.append(self.logits.cpu().numpy().copy())
            if t == n_decode:
                break
            if forced is not None:
                tk = np.ascontiguousarray(forced[:, t:t + 1], dtype=np.int32)
                self.step(tb.DECODE, tk, 1)
                toks.append(tk[:, 0].copy())
            else:
                self.compute.synchronize()
                toks.append(self.argmax.cpu().numpy().copy())
                self.step(tb.DECODE, None, 1)
        self.sync()
        return out, (np.stack(toks, axis=1) if toks else np.zeros((self.cfg.B, 0), np.int32))

    def capture_run(self, prompt_pinned, n_decode: int):
        """Captures prefill + n_decode free-running decode steps into one CUDA graph (dense models).  prompt_pinned:
        int32 host tensor/array [B, S] that stays alive and unchanged while the graph is replayed."""
        self._prompt_keep = prompt_pinned
        arr = prompt_pinned.numpy() if hasattr(prompt_pinned, "numpy") else prompt_pinned
        self.reset()
        self.s.ctx.run_capture_begin(self.compute, self.copy)
        try:
            self.step(tb.PREFILL, arr, arr.shape[1])
            for _ in range(n_decode):
                self.step(tb.DECODE, None, 1)
        finally:
            self.s.ctx.run_capture_end()

    def replay(self):
        self.s.ctx.run_graph_launch(self.compute)
