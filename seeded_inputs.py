"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This module holds the *workload*, and none of the method's arithmetic: the five
model shapes, the sub-allocation layout of the host pool (which tensor sits at
which pool offset), the counter-based weight generator, the prompts and the MoE
router bias.  Neither the forward pass, nor the op trace, nor the prefetch policy
live here; the oracle and the library each implement those on their own.

Recipe (all integer arithmetic apart from one fp32 multiply, so any two IEEE
machines produce the same bits):

* ``h = splitmix64(seed ^ (role_id << 40) ^ element_index)`` with
  ``element_index = row * cols + col`` of the ``[out, in]`` matrix;
* split ``h`` into four 16-bit lanes, ``s = u0+u1+u2+u3 - 131070`` (Irwin-Hall,
  variance ``4 * (65536**2 - 1) / 12``), ``w = bf16_rne(float32(s) * c)`` with
  ``c = float32(0.02 / (65536 * sqrt(1/3)))``: mean 0, std 0.02;
* norm gains are exactly 1.0 (a N(0, 0.02) gain would wipe out the signal);
* ``token[b, p] = splitmix64(seed ^ 0x70726f6d ^ (b << 32) ^ p) mod V``.

The paper evaluates ten public LLM checkpoints at an oversubscription factor of
2.0; their weights and prompts are not available here, so these seeded shapes of
the same family (Llama-/Mixtral-style decoders) stand in for them.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np

U64 = np.uint64
MASK64 = (1 << 64) - 1

# tensor kinds (also the role ids used in the weight hash)
K_EMBED, K_G1, K_WQ, K_WK, K_WV, K_WO, K_G2, K_WG, K_WU, K_WD, K_GF, K_LM, K_ROUTER, K_KT, K_VT = range(15)
KIND_NAMES = ["embed", "g1", "wq", "wk", "wv", "wo", "g2", "wg", "wu", "wd", "gf", "lm_head",
              "router", "k_tile", "v_tile"]
F_READONLY, F_MUTABLE = 1, 2
POOL_ALIGN = 512          # sub-allocation granularity of the pool
BASE_SEED = 0x2609061720


def splitmix64_int(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & MASK64
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
    return z ^ (z >> 31)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """Vectorised splitmix64 finaliser over a uint64 array (wraps mod 2**64)."""
    with np.errstate(over="ignore"):
        z = x + U64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> U64(30))) * U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> U64(27))) * U64(0x94D049BB133111EB)
        return z ^ (z >> U64(31))


_C_SCALE = np.float32(0.02 / (65536.0 * math.sqrt(1.0 / 3.0)))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_bits_range(seed: int, role: int, start: int, count: int) -> np.ndarray:
    idx = np.arange(start, start + count, dtype=U64)
    h = splitmix64(idx ^ U64((seed ^ (role << 40)) & MASK64))
    s = ((h & U64(0xFFFF)) + ((h >> U64(16)) & U64(0xFFFF)) + ((h >> U64(32)) & U64(0xFFFF))
         + (h >> U64(48))).astype(np.int64) - 131070
    return f32_to_bf16_bits(s.astype(np.float32) * _C_SCALE)


def normal_bf16_bits(seed: int, role: int, start: int, count: int, out: Optional[np.ndarray] = None,
                     threads: int = 8) -> np.ndarray:
    """bf16 bit patterns of elements [start, start+count) of the tensor stream ``role``."""
    if out is None:
        out = np.empty(count, dtype=np.uint16)
    chunk = 1 << 22
    if count <= chunk:
        out[:count] = _normal_bits_range(seed, role, start, count)
        return out
    spans = [(o, min(chunk, count - o)) for o in range(0, count, chunk)]

    def work(sp):
        o, n = sp
        out[o:o + n] = _normal_bits_range(seed, role, start + o, n)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(work, spans))
    return out


def weight_role(kind: int, layer: int, expert: int) -> int:
    """Role id of one logical weight matrix (< 2**24, so ``role << 40`` stays inside 64 bits)."""
    return (kind << 16) | ((layer + 1) << 4) | (expert + 1)


@dataclass(frozen=True)
class ModelConfig:
    name: str
    L: int
    d: int
    Hq: int
    Hkv: int
    Dh: int
    F: int
    V: int
    B: int
    S: int            # prompt tokens
    T: int            # decode steps
    TK: int           # tokens per KV tile
    E: int = 0        # experts (0 = dense FFN)
    topk: int = 0
    seed: int = BASE_SEED
    budget_rule: str = ""      # "half_w_kv" | "half_w" | "<bytes>"
    rope_base: float = 10000.0
    eps: float = 1e-5
    zipf_s: float = 1.2

    @property
    def max_len(self) -> int:
        return self.S + self.T

    @property
    def n_tiles(self) -> int:
        return (self.max_len + self.TK - 1) // self.TK


CONFIGS: Dict[int, ModelConfig] = {
    1: ModelConfig("tiny", 4, 256, 4, 4, 64, 1024, 4096, 1, 32, 16, 16, seed=BASE_SEED + 1, budget_rule="half_w_kv"),
    2: ModelConfig("llama1b", 16, 2048, 32, 8, 64, 8192, 32000, 1, 512, 128, 128, seed=BASE_SEED + 2, budget_rule="half_w"),
    3: ModelConfig("llama8b", 32, 4096, 32, 8, 128, 14336, 128256, 8, 1024, 256, 256, seed=BASE_SEED + 3, budget_rule=str(8 << 30)),
    4: ModelConfig("llama70b", 80, 8192, 64, 8, 128, 28672, 128256, 16, 2048, 64, 64, seed=BASE_SEED + 4, budget_rule=str(64 << 30)),
    5: ModelConfig("mixtral", 32, 4096, 32, 8, 128, 14336, 32000, 32, 512, 128, 128, E=8, topk=2, seed=BASE_SEED + 5, budget_rule=str(40 << 30)),
}


def reduced_tokens(cfg: ModelConfig, B: int = 1, S: int = 16, T: int = 4, TK: Optional[int] = None) -> ModelConfig:
    """Same widths and depth, fewer tokens: the case a CPU forward pass finishes in minutes."""
    tk = TK if TK is not None else min(cfg.TK, 4)
    return replace(cfg, name=cfg.name + "_reduced", B=B, S=S, T=T, TK=tk)


@dataclass
class TensorSpec:
    """One registered sub-range of the pool."""
    tid: int
    kind: int
    layer: int          # -1 for model-level tensors
    expert: int         # -1 unless an expert weight
    block: int          # out-row block index (weights) or tile index (KV)
    row0: int
    rows: int
    cols: int
    elem_bytes: int
    pool_off: int
    size: int
    flags: int
    site_hash: int

    @property
    def name(self) -> str:
        s = KIND_NAMES[self.kind]
        if self.layer >= 0:
            s += f".l{self.layer}"
        if self.expert >= 0:
            s += f".e{self.expert}"
        return s + f".b{self.block}"


@dataclass
class PoolLayout:
    cfg: ModelConfig
    tensors: List[TensorSpec]
    pool_bytes: int
    weight_bytes: int       # sum of registered weight sizes (no padding)
    kv_bytes: int
    budget: int
    sub_range_cap: int
    by_role: Dict[tuple, List[TensorSpec]] = field(default_factory=dict)

    def blocks(self, kind: int, layer: int = -1, expert: int = -1) -> List[TensorSpec]:
        return self.by_role[(kind, layer, expert)]


def _align(x: int, a: int = POOL_ALIGN) -> int:
    return (x + a - 1) // a * a


def sub_range_cap(budget: int) -> int:
    """Largest power of two <= budget/8, clamped to [128 KiB, 32 MiB].  (32 MiB copies already run at the link's
    full rate; larger blocks only enlarge the staging ring, which is sized as two of them, at the expense of pins.
    Below that, a block must be large enough for its copy to outlast the kernel that consumes the block before it plus
    the hand-over between the two streams: with a ring of two blocks the next copy cannot start earlier.  Measured on the
    tiny configuration: 128 KiB blocks - 35 copies and 96 launches per decode step - reach 0.24 of the step roofline,
    512 KiB blocks - 11 copies, 50 launches - 0.58.)"""
    c = 1 << max(0, (budget // 8).bit_length() - 1)
    return max(128 << 10, min(32 << 20, c))


def block_rows(rows: int, cols: int, cap: int) -> int:
    rpb = max(1, cap // (cols * 2))
    if rpb >= 128:
        rpb -= rpb % 128
    return min(rows, rpb)


def weight_matrices(cfg: ModelConfig):
    """(kind, layer, expert, rows(out), cols(in)) in sub-allocation order; norm gains have rows=1."""
    qd, kvd = cfg.Hq * cfg.Dh, cfg.Hkv * cfg.Dh
    out = [(K_EMBED, -1, -1, cfg.V, cfg.d)]
    for l in range(cfg.L):
        out += [(K_G1, l, -1, 1, cfg.d), (K_WQ, l, -1, qd, cfg.d), (K_WK, l, -1, kvd, cfg.d),
                (K_WV, l, -1, kvd, cfg.d), (K_WO, l, -1, cfg.d, qd), (K_G2, l, -1, 1, cfg.d)]
        if cfg.E == 0:
            out += [(K_WG, l, -1, cfg.F, cfg.d), (K_WU, l, -1, cfg.F, cfg.d), (K_WD, l, -1, cfg.d, cfg.F)]
        else:
            out += [(K_ROUTER, l, -1, cfg.E, cfg.d)]
            for e in range(cfg.E):
                out += [(K_WG, l, e, cfg.F, cfg.d), (K_WU, l, e, cfg.F, cfg.d), (K_WD, l, e, cfg.d, cfg.F)]
    out += [(K_GF, -1, -1, 1, cfg.d), (K_LM, -1, -1, cfg.V, cfg.d)]
    return out


def build_layout(cfg: ModelConfig, budget: Optional[int] = None, cap: Optional[int] = None) -> PoolLayout:
    """Sub-allocate every weight (block) and KV tile of ``cfg`` in one pool, 512-byte aligned."""
    mats = weight_matrices(cfg)
    w_bytes = sum(r * c * 2 for (_, _, _, r, c) in mats)
    tile_bytes = cfg.B * cfg.Hkv * cfg.TK * cfg.Dh * 2
    kv_bytes = cfg.L * 2 * cfg.n_tiles * tile_bytes
    if budget is None:
        if cfg.budget_rule == "half_w_kv":
            budget = (w_bytes + kv_bytes) // 2
        elif cfg.budget_rule == "half_w":
            budget = w_bytes // 2
        else:
            budget = int(cfg.budget_rule)
    if cap is None:
        cap = sub_range_cap(budget)
    tensors: List[TensorSpec] = []
    off = 0

    def add(kind, layer, expert, block, row0, rows, cols, flags):
        nonlocal off
        size = rows * cols * 2
        t = TensorSpec(len(tensors), kind, layer, expert, block, row0, rows, cols, 2, off, size, flags,
                       splitmix64_int(0xA110C000 + kind))
        tensors.append(t)
        off = _align(off + size)

    for (kind, layer, expert, rows, cols) in mats:
        if kind in (K_EMBED, K_G1, K_G2, K_GF, K_ROUTER):
            add(kind, layer, expert, 0, 0, rows, cols, F_READONLY)      # gather table / small: one tensor
            continue
        rpb = block_rows(rows, cols, cap)
        for b, r0 in enumerate(range(0, rows, rpb)):
            add(kind, layer, expert, b, r0, min(rpb, rows - r0), cols, F_READONLY)
    for l in range(cfg.L):
        for kind in (K_KT, K_VT):
            for j in range(cfg.n_tiles):
                add(kind, l, -1, j, j * cfg.TK, cfg.B * cfg.Hkv * cfg.TK, cfg.Dh, F_MUTABLE)
    lay = PoolLayout(cfg, tensors, off, w_bytes, kv_bytes, budget, cap)
    for t in tensors:
        lay.by_role.setdefault((t.kind, t.layer, t.expert), []).append(t)
    return lay


def fill_tensor(cfg: ModelConfig, t: TensorSpec, out: np.ndarray) -> None:
    """Write tensor ``t``'s bf16 bits into ``out`` (uint16 view of its pool range)."""
    n = t.rows * t.cols
    if t.kind in (K_G1, K_G2, K_GF):
        out[:n] = 0x3F80                       # bf16 1.0
    elif t.kind in (K_KT, K_VT):
        out[:n] = 0
    else:
        normal_bf16_bits(cfg.seed, weight_role(t.kind, t.layer, t.expert), t.row0 * t.cols, n, out=out)


def fill_pool(lay: PoolLayout, pool_u8: np.ndarray) -> None:
    """Materialise every tensor of the layout into a caller-owned byte buffer of ``lay.pool_bytes``."""
    u16 = pool_u8.view(np.uint16)
    for t in lay.tensors:
        fill_tensor(lay.cfg, t, u16[t.pool_off // 2: t.pool_off // 2 + t.rows * t.cols])


def _torch_normal_bits(seed: int, role: int, start: int, count: int, device):
    """Same stream as normal_bf16_bits(), evaluated with torch integer ops (int64 wraps like uint64; logical
    right shifts are emulated by masking).  Returns an int16 tensor of bf16 bit patterns on `device`."""
    import torch

    def sgn(v):                       # two's-complement view of a uint64 constant
        v &= MASK64
        return v - (1 << 64) if v >= (1 << 63) else v

    def lsr(z, k):
        return (z >> k) & ((1 << (64 - k)) - 1)

    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    z = (idx ^ sgn(seed ^ (role << 40))) + sgn(0x9E3779B97F4A7C15)
    z = (z ^ lsr(z, 30)) * sgn(0xBF58476D1CE4E5B9)
    z = (z ^ lsr(z, 27)) * sgn(0x94D049BB133111EB)
    h = z ^ lsr(z, 31)
    s = (h & 0xFFFF) + (lsr(h, 16) & 0xFFFF) + (lsr(h, 32) & 0xFFFF) + lsr(h, 48) - 131070
    w = (s.to(torch.float32) * float(_C_SCALE)).to(torch.bfloat16)
    return w.view(torch.int16)


def fill_pool_torch(lay: PoolLayout, pool_u8, device="cuda:0", chunk: int = 1 << 26) -> None:
    """fill_pool() for large pools: generates on `device` and copies into the (pinned) torch uint8 pool tensor.
    Bit-identical to the numpy path (tested)."""
    import torch
    i16 = pool_u8.view(torch.int16)
    for t in lay.tensors:
        n = t.rows * t.cols
        dst = i16[t.pool_off // 2: t.pool_off // 2 + n]
        if t.kind in (K_G1, K_G2, K_GF):
            dst.fill_(0x3F80)
        elif t.kind in (K_KT, K_VT):
            dst.zero_()
        else:
            role = weight_role(t.kind, t.layer, t.expert)
            for o in range(0, n, chunk):
                c = min(chunk, n - o)
                dst[o:o + c].copy_(_torch_normal_bits(lay.cfg.seed, role, t.row0 * t.cols + o, c, device))
    if str(device).startswith("cuda"):
        torch.cuda.synchronize()


def weights_as_bits(lay: PoolLayout) -> Dict[tuple, np.ndarray]:
    """Whole logical matrices (blocks re-joined) as bf16 bit arrays ``[rows, cols]``, keyed (kind, layer, expert)."""
    out = {}
    for (kind, layer, expert, rows, cols) in weight_matrices(lay.cfg):
        a = np.empty(rows * cols, dtype=np.uint16)
        if kind in (K_G1, K_G2, K_GF):
            a[:] = 0x3F80
        else:
            normal_bf16_bits(lay.cfg.seed, weight_role(kind, layer, expert), 0, rows * cols, out=a)
        out[(kind, layer, expert)] = a.reshape(rows, cols)
    return out


def prompt_tokens(cfg: ModelConfig) -> np.ndarray:
    b = np.arange(cfg.B, dtype=U64)[:, None]
    p = np.arange(cfg.S, dtype=U64)[None, :]
    h = splitmix64(U64((cfg.seed ^ 0x70726F6D) & MASK64) ^ (b << U64(32)) ^ p)
    return (h % U64(cfg.V)).astype(np.int32)


def router_bias(cfg: ModelConfig) -> np.ndarray:
    """fp32 ``[L, E]`` router bias: ln of a Zipf(s) law over a seeded per-layer permutation of the experts."""
    if cfg.E == 0:
        return np.zeros((cfg.L, 0), dtype=np.float32)
    p = np.array([r ** (-cfg.zipf_s) for r in range(1, cfg.E + 1)], dtype=np.float64)
    p /= p.sum()
    out = np.empty((cfg.L, cfg.E), dtype=np.float32)
    for l in range(cfg.L):
        keys = [splitmix64_int((cfg.seed ^ 0x7A697066 ^ (l << 8) ^ e) & MASK64) for e in range(cfg.E)]
        rank = np.argsort(np.array(keys, dtype=np.uint64), kind="stable")      # expert rank[r] gets popularity r
        for r, e in enumerate(rank):
            out[l, e] = np.float32(math.log(p[r]))
    return out
