"""Oracle op trace: the ordered list of (kernel, tensor) access pairs with analytic costs.

TEST INFRASTRUCTURE - see oracle/__init__.py.

The paper records kernel-tensor access pairs in one offline profiling pass (Section IV-D,
"Kernel-Tensor Access Tracing") and counts FLOPs and loads per kernel by binary
instrumentation (Section IV-G).  Here the counts are analytic functions of the shapes,
fixed in one table below; the trace is logical (one op per weight block, whatever the
GPU fuses).  All quantities are Python integers.

Per step with M = B*q tokens, pos0 cached tokens before the step, kvlen = pos0 + q:

  embed      flops 0                       hbm M*d*6                         embed R, touched M*d*2
  rmsnorm    flops 4*m*d                   hbm m*d*6 + 2*d                   gain R, touched 2*d
  gemm block flops 2*m*K*n                 hbm 2*m*K + 2*K*n + 4*m*n (+4*m*n residual)   block R, touched size
  rope+kv    flops 6*M*(Hq+Hkv)*Dh         hbm M*(Hq+2*Hkv)*Dh*6             K tiles then V tiles of the new tokens, W
  attention  flops 4*B*Hq*Dh*(tri(kvlen)-tri(pos0))   hbm 4*M*Hq*Dh + 4*B*Hkv*kvlen*Dh    K tiles then V tiles with valid tokens, R
  swiglu     flops 8*m*F                   hbm m*F*10                        -
  router     flops 2*M*d*E                 hbm 2*M*d + 2*d*E + 4*M*E         router R, touched size
  argmax     flops B*V                     hbm 4*B*V + 4*B                   -
with tri(n) = n*(n+1)/2.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

OP_EMBED, OP_RMSNORM, OP_GEMM, OP_ROPE_KV, OP_ATTN, OP_SWIGLU, OP_ROUTER, OP_ARGMAX = range(8)
MODE_R, MODE_W, MODE_RW = 1, 2, 3
STEP_PREFILL, STEP_DECODE = 0, 1
# tensor kinds of the layout (literal copies: the oracle depends on the layout's numbers, not its code)
K_EMBED, K_G1, K_WQ, K_WK, K_WV, K_WO, K_G2, K_WG, K_WU, K_WD, K_GF, K_LM, K_ROUTER, K_KT, K_VT = range(15)


@dataclass
class Op:
    step: int
    site: int
    layer: int
    kind: int
    flops: int
    hbm: int
    acc: List[Tuple[int, int, int]] = field(default_factory=list)     # (tensor id, mode, touched bytes)
    m: int = 0                                                          # rows the op processes (not exported)
    expert: int = -1


def site_of(kind: int, sub: int) -> int:
    return (kind << 8) | sub


def tri(n: int) -> int:
    return n * (n + 1) // 2


def step_ops(lay, step: int, q: int, pos0: int, expert_counts=None) -> List[Op]:
    """Ops of one forward step.  expert_counts[l][e] = tokens routed to expert e (MoE only)."""
    cfg = lay.cfg
    B, d, Hq, Hkv, Dh, F, V, TK = cfg.B, cfg.d, cfg.Hq, cfg.Hkv, cfg.Dh, cfg.F, cfg.V, cfg.TK
    M = B * q
    kvlen = pos0 + q
    ops: List[Op] = []

    def gemm_blocks(kind, layer, expert, m, residual):
        for t in lay.blocks(kind, layer, expert):
            K, n = t.cols, t.rows
            hbm = 2 * m * K + 2 * K * n + 4 * m * n + (4 * m * n if residual else 0)
            ops.append(Op(step, site_of(OP_GEMM, kind), layer, OP_GEMM, 2 * m * K * n, hbm,
                          [(t.tid, MODE_R, t.size)], m, expert))

    def norm(kind, layer, m):
        g = lay.blocks(kind, layer)[0]
        ops.append(Op(step, site_of(OP_RMSNORM, kind), layer, OP_RMSNORM, 4 * m * d, m * d * 6 + 2 * d,
                      [(g.tid, MODE_R, 2 * d)], m))

    emb = lay.blocks(K_EMBED)[0]
    ops.append(Op(step, site_of(OP_EMBED, 0), -1, OP_EMBED, 0, M * d * 6, [(emb.tid, MODE_R, M * d * 2)], M))
    for l in range(cfg.L):
        norm(K_G1, l, M)
        gemm_blocks(K_WQ, l, -1, M, False)
        gemm_blocks(K_WK, l, -1, M, False)
        gemm_blocks(K_WV, l, -1, M, False)
        kt, vt = lay.blocks(K_KT, l), lay.blocks(K_VT, l)
        acc = []
        for tiles in (kt, vt):
            for j in range(pos0 // TK, (kvlen - 1) // TK + 1):
                ntok = min(kvlen, (j + 1) * TK) - max(pos0, j * TK)
                acc.append((tiles[j].tid, MODE_W, B * Hkv * ntok * Dh * 2))
        ops.append(Op(step, site_of(OP_ROPE_KV, 0), l, OP_ROPE_KV, 6 * M * (Hq + Hkv) * Dh,
                      M * (Hq + 2 * Hkv) * Dh * 6, acc, M))
        acc = []
        for tiles in (kt, vt):
            for j in range(0, (kvlen - 1) // TK + 1):
                valid = min(kvlen, (j + 1) * TK) - j * TK
                acc.append((tiles[j].tid, MODE_R, B * Hkv * valid * Dh * 2))
        ops.append(Op(step, site_of(OP_ATTN, 0), l, OP_ATTN, 4 * B * Hq * Dh * (tri(kvlen) - tri(pos0)),
                      4 * M * Hq * Dh + 4 * B * Hkv * kvlen * Dh, acc, M))
        gemm_blocks(K_WO, l, -1, M, True)
        norm(K_G2, l, M)
        if cfg.E == 0:
            gemm_blocks(K_WG, l, -1, M, False)
            gemm_blocks(K_WU, l, -1, M, False)
            ops.append(Op(step, site_of(OP_SWIGLU, 0), l, OP_SWIGLU, 8 * M * F, M * F * 10, [], M))
            gemm_blocks(K_WD, l, -1, M, True)
        else:
            r = lay.blocks(K_ROUTER, l)[0]
            ops.append(Op(step, site_of(OP_ROUTER, 0), l, OP_ROUTER, 2 * M * d * cfg.E,
                          2 * M * d + 2 * d * cfg.E + 4 * M * cfg.E, [(r.tid, MODE_R, r.size)], M))
            for e in range(cfg.E):
                me = int(expert_counts[l][e])
                if me == 0:
                    continue
                gemm_blocks(K_WG, l, e, me, False)
                gemm_blocks(K_WU, l, e, me, False)
                ops.append(Op(step, site_of(OP_SWIGLU, 0), l, OP_SWIGLU, 8 * me * F, me * F * 10, [], me, e))
                gemm_blocks(K_WD, l, e, me, True)
    norm(K_GF, -1, B)
    gemm_blocks(K_LM, -1, -1, B, False)
    ops.append(Op(step, site_of(OP_ARGMAX, 0), -1, OP_ARGMAX, B * V, 4 * B * V + 4 * B, [], B))
    return ops


def run_trace(lay, expert_counts=None, n_decode=None) -> Tuple[List[Op], List[Tuple[int, int, int]]]:
    """Whole run: prefill of S tokens, then T decode steps.
    Returns (ops, steps) with steps[k] = (step kind, first op index, op count)."""
    cfg = lay.cfg
    T = cfg.T if n_decode is None else n_decode
    ops: List[Op] = []
    steps = []
    for k in range(1 + T):
        q, pos0 = (cfg.S, 0) if k == 0 else (1, cfg.S + k - 1)
        so = step_ops(lay, k, q, pos0, None if expert_counts is None else expert_counts[k])
        steps.append((STEP_PREFILL if k == 0 else STEP_DECODE, len(ops), len(so)))
        ops += so
    return ops, steps
