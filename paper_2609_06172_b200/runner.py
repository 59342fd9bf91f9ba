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
