"""ctypes binding of libtgp.so: the same names as include/tgp.h, argument marshalling only.

Every step of the path runs inside the library.  If the library is missing this module raises:
there is no Python or CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libtgp.so")

OK, E_INVAL, E_OVERLAP, E_RANGE, E_UNKNOWN_TENSOR, E_BUDGET_TOO_SMALL, E_NO_PLAN, E_CUDA, E_MISMATCH, E_STATE, E_TOO_LARGE = \
    0, -1, -2, -3, -4, -5, -6, -7, -8, -9, -10
POOL_PINNED, POOL_MANAGED, POOL_PLAIN = 1, 2, 4
T_READONLY, T_MUTABLE = 1, 2
R, W = 1, 2
PREFILL, DECODE = 0, 1
VAR_EXPLICIT_RING, VAR_MANAGED_HINTS, VAR_MANAGED_DEMAND, VAR_MANAGED_OBJECT = 0, 1, 2, 3
BIT_A, BIT_P, BIT_ZC, BIT_W = 1, 2, 4, 8
X_CLASSES, X_TENSORS, X_PINS, X_COMMANDS, X_TOTALS = range(5)
X_TAIL = 0x100
# tensor kinds (TGP_K_*)
(K_EMBED, K_G1, K_WQ, K_WK, K_WV, K_WO, K_G2, K_WG, K_WU, K_WD, K_GF, K_LM, K_ROUTER, K_KTILE, K_VTILE) = range(15)
TAP_H, TAP_HF, TAP_Q, TAP_KTILE, TAP_VTILE, TAP_O, TAP_A = range(7)


class Machine(C.Structure):
    _fields_ = [("peak_flops", C.c_uint64), ("hbm_Bps", C.c_uint64), ("h2d_Bps", C.c_uint64), ("d2h_Bps", C.c_uint64)]


class Access(C.Structure):
    _fields_ = [("tensor", C.c_uint32), ("mode", C.c_uint32), ("touched_bytes", C.c_uint64)]


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("L", "d", "Hq", "Hkv", "Dh", "F", "V", "E", "topk", "B", "max_len", "TK")] + \
               [("rope_base", C.c_float), ("eps", C.c_float)]


class RoleEntry(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("layer", C.c_int32), ("expert", C.c_int32), ("block", C.c_uint32),
                ("row0", C.c_uint32), ("rows", C.c_uint32), ("tensor", C.c_uint32)]


class StepStats(C.Structure):
    _fields_ = [("h2d_bytes", C.c_uint64), ("d2h_bytes", C.c_uint64), ("zc_bytes", C.c_uint64),
                ("n_cmds", C.c_uint32), ("n_launches", C.c_uint32), ("n_mismatch", C.c_uint32), ("step_ms", C.c_float)]


class TgpError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        super().__init__(f"{where}: {lib().tgp_strerror(code).decode()} ({code}) {detail}")


_lib = None
_P, _U32, _U64, _I32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int32
_SIGS = {
    "tgp_create": [C.POINTER(_P), C.POINTER(Machine)],
    "tgp_destroy": [_P],
    "tgp_pool_register": [_P, _P, _U64, _U32, C.POINTER(_U32)],
    "tgp_tensor_register": [_P, _U32, _U64, _U64, _U64, _I32, _U32, _U32, C.POINTER(_U32)],
    "tgp_tensor_lookup": [_P, _P, C.POINTER(_U32), C.POINTER(_U64)],
    "tgp_tensor_identity": [_P, _U32, C.POINTER(_U64), C.POINTER(_U64)],
    "tgp_trace_begin": [_P],
    "tgp_trace_step": [_P, _U32],
    "tgp_trace_op": [_P, _U64, _I32, _U32, _U64, _U64, _U32, C.POINTER(Access)],
    "tgp_trace_end": [_P],
    "tgp_model_trace": [_P, _U32, _U32, C.POINTER(_U32)],
    "tgp_trace_export": [_P, _P, C.POINTER(_U64)],
    "tgp_set_budget": [_P, _U64],
    "tgp_set_variant": [_P, _U32, _U32],
    "tgp_set_object_bytes": [_P, _U64],
    "tgp_set_measured_times": [_P, C.POINTER(_U64), _U64],
    "tgp_plan": [_P],
    "tgp_replan_begin": [_P, _U32, C.POINTER(_U64), _U64],
    "tgp_replan_wait": [_P],
    "tgp_replan_commit": [_P],
    "tgp_set_replan_keep": [C.c_void_p, C.c_int],
    "tgp_plan_export": [_P, _U32, _P, C.POINTER(_U64)],
    "tgp_set_arena": [_P, _P, _U64],
    "tgp_model_workspace_bytes": [C.POINTER(ModelCfg), _U32, C.POINTER(_U64)],
    "tgp_model_bind": [_P, C.POINTER(ModelCfg), C.POINTER(RoleEntry), _U32, _P, _P, _U64, _U32],
    "tgp_run_reset": [_P],
    "tgp_step": [_P, _U32, _P, _U32, _U32, _P, _P, _P, _P, C.POINTER(StepStats)],
    "tgp_expert_counts": [_P, C.POINTER(_U32), C.POINTER(_U64)],
    "tgp_managed_alloc": [C.POINTER(_P), _U64],
    "tgp_managed_free": [_P],
    "tgp_managed_evict": [_P, _U64],
    "tgp_run_capture_begin": [_P, _P, _P],
    "tgp_run_capture_end": [_P],
    "tgp_run_graph_launch": [_P, _P],
    "tgp_set_tap": [_P, _P, _U64],
    "tgp_tap_index": [_P, C.POINTER(_U64), C.POINTER(_U64)],
    "tgp_set_op_timing": [_P, C.c_int],
    "tgp_op_times": [_P, C.POINTER(C.c_float), _U32, C.POINTER(_U32), C.POINTER(_U32)],
    "tgp_k_embed": [_P, _P, _P, _U32, _U32, _U32, _P],
    "tgp_k_embed_status": [C.POINTER(C.c_int), C.POINTER(_U32), C.POINTER(C.c_int32)],
    "tgp_k_status_clear": [],
    "tgp_k_wait_test": [_U64, C.c_int],
    "tgp_k_rmsnorm": [_P, _U32, _P, _P, _U32, _U32, C.c_float, _P],
    "tgp_k_gemm": [_P, _P, _P, _U32, _U32, _U32, _U32, _U32, C.c_int, _P],
    "tgp_k_gemm_group": [_P, _U32, _P, _P, C.POINTER(_U32), C.POINTER(_U32), _U32, _U32, C.c_int, _P],
    "tgp_k_gemm_group_key": [_U32, _U32, _U32, C.POINTER(_U32)],
    "tgp_k_gemm_group_select": [C.c_int],
    "tgp_k_gemm_last_kernel": [C.c_char_p, _U32],
    "tgp_k_gemm_select": [C.c_int],
    "tgp_k_decode_fuse": [C.c_int],
    "tgp_k_merge_copies": [C.c_int],
    "tgp_copies_issued": [_P, C.POINTER(_U64)],
    "tgp_k_swiglu_epilogue": [C.c_int],
    "tgp_k_attn_select": [C.c_int],
    "tgp_k_attn_decode_select": [C.c_int],
    "tgp_k_gemv_overlap": [C.c_int],
    "tgp_k_gemm_chain": [C.c_int],
    "tgp_k_skinny_select": [C.c_int],
    "tgp_k_gemm_tc_variant": [C.c_int],
    "tgp_k_gemm_status": [C.POINTER(C.c_int)],
    "tgp_k_attn_status": [C.POINTER(C.c_int)],
    "tgp_k_rope_tables": [_U32, _U32, C.c_float, _P, _P],
    "tgp_k_rope_kv": [_P, _P, _P, _P, C.POINTER(_P), C.POINTER(_P), _U32, _P, _P, C.POINTER(ModelCfg), _U32, _U32, _U32, _P],
    "tgp_k_attn": [_P, C.POINTER(_P), C.POINTER(_P), _U32, _P, C.POINTER(ModelCfg), _U32, _U32, _U32, _P, _P],
    "tgp_k_attn_decode_static": [_P, C.POINTER(_P), C.POINTER(_P), _U32, _P, C.POINTER(ModelCfg), _U32, _U32, _P],
    "tgp_k_attn_scratch_bytes": [C.POINTER(ModelCfg), C.POINTER(_U64)],
    "tgp_k_swiglu": [_P, _P, _P, _U64, _P],
    "tgp_k_argmax": [_P, _P, _U32, _U32, _P],
}


def lib():
    """The loaded library; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_06172_b200.build` "
                              "(the hot path has no Python or CPU fallback)")
        l = C.CDLL(LIB_PATH)
        for name, args in _SIGS.items():
            f = getattr(l, name)
            f.argtypes = args
            f.restype = None if name == "tgp_destroy" else C.c_int
        l.tgp_strerror.argtypes, l.tgp_strerror.restype = [C.c_int], C.c_char_p
        l.tgp_last_error.argtypes, l.tgp_last_error.restype = [_P], C.c_char_p
        _lib = l
    return _lib


def exported_symbols():
    return sorted(list(_SIGS) + ["tgp_strerror", "tgp_last_error"])


def parse_trace(blob):
    """Decodes the blob of tgp_trace_export(): per op u32 step, u64 site, i32 layer, u32 kind, u64 flops, u64 hbm bytes,
    u32 n_acc, then n_acc x (u32 tensor, u32 mode, u64 touched).  Returns a list of
    (step, site, layer, kind, flops, hbm, [(tensor, mode, touched)])."""
    import struct
    ops, off = [], 0
    head = struct.Struct("<IQiIQQI")
    while off < len(blob):
        step, site, layer, kind, flops, hbm, n = head.unpack_from(blob, off)
        off += head.size
        acc = [struct.unpack_from("<IIQ", blob, off + 16 * k) for k in range(n)]
        off += 16 * n
        ops.append((step, site, layer, kind, flops, hbm, acc))
    return ops


def _ptr(x):
    """Address of a numpy array / torch tensor / int / None as a void pointer value."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "cuda_stream"):
        return x.cuda_stream
    raise TypeError(type(x))


class Ctx:
    """One tgp_ctx.  Methods carry the C names without the prefix; each raises TgpError on a negative code."""

    def __init__(self, peak_flops, hbm_Bps, h2d_Bps, d2h_Bps):
        self._h = _P()
        m = Machine(peak_flops, hbm_Bps, h2d_Bps, d2h_Bps)
        rc = lib().tgp_create(C.byref(self._h), C.byref(m))
        if rc:
            raise TgpError(rc, "tgp_create")
        self._keep = []

    def close(self):
        if self._h:
            lib().tgp_destroy(self._h)
            self._h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, rc, where):
        if rc:
            raise TgpError(rc, where, lib().tgp_last_error(self._h).decode())
        return rc

    def pool_register(self, host_base, nbytes, flags):
        out = _U32()
        self._ck(lib().tgp_pool_register(self._h, _ptr(host_base), nbytes, flags, C.byref(out)), "tgp_pool_register")
        self._keep.append(host_base)
        return out.value

    def tensor_register(self, pool, offset, nbytes, site_hash, layer, kind, flags):
        out = _U32()
        self._ck(lib().tgp_tensor_register(self._h, pool, offset, nbytes, site_hash, layer, kind, flags, C.byref(out)), "tgp_tensor_register")
        return out.value

    def tensor_lookup(self, host_addr):
        t, o = _U32(), _U64()
        self._ck(lib().tgp_tensor_lookup(self._h, host_addr, C.byref(t), C.byref(o)), "tgp_tensor_lookup")
        return t.value, o.value

    def tensor_identity(self, tid):
        s, c = _U64(), _U64()
        self._ck(lib().tgp_tensor_identity(self._h, tid, C.byref(s), C.byref(c)), "tgp_tensor_identity")
        return s.value, c.value

    def trace_begin(self):
        self._ck(lib().tgp_trace_begin(self._h), "tgp_trace_begin")

    def trace_step(self, kind):
        self._ck(lib().tgp_trace_step(self._h, kind), "tgp_trace_step")

    def trace_op(self, site, layer, kind, flops, hbm, acc):
        arr = (Access * max(1, len(acc)))(*[Access(t, m, b) for (t, m, b) in acc])
        self._ck(lib().tgp_trace_op(self._h, site, layer, kind, flops, hbm, len(acc), arr), "tgp_trace_op")

    def trace_end(self):
        self._ck(lib().tgp_trace_end(self._h), "tgp_trace_end")

    def model_trace(self, S, T, expert_counts=None):
        p = None
        if expert_counts is not None:
            ec = np.ascontiguousarray(expert_counts, dtype=np.uint32)
            p = ec.ctypes.data_as(C.POINTER(_U32))
        self._ck(lib().tgp_model_trace(self._h, S, T, p), "tgp_model_trace")

    def trace_export(self):
        n = _U64()
        self._ck(lib().tgp_trace_export(self._h, None, C.byref(n)), "tgp_trace_export")
        buf = C.create_string_buffer(max(1, n.value))
        self._ck(lib().tgp_trace_export(self._h, buf, C.byref(n)), "tgp_trace_export")
        return buf.raw[:n.value]

    def trace_ops(self):
        """The recorded trace decoded: a list of (step, site, layer, kind, flops, hbm bytes, [(tensor, mode, touched)])."""
        return parse_trace(self.trace_export())

    def copies_issued(self):
        n = _U64()
        self._ck(lib().tgp_copies_issued(self._h, C.byref(n)), "tgp_copies_issued")
        return n.value

    def replan_begin(self, first_step, op_ns=None):
        """Starts planning the steps from first_step on (helper thread); op_ns: uint64 per op of the whole trace, or None."""
        if op_ns is None:
            self._ck(lib().tgp_replan_begin(self._h, first_step, None, 0), "tgp_replan_begin")
        else:
            a = np.ascontiguousarray(op_ns, dtype=np.uint64)
            self._ck(lib().tgp_replan_begin(self._h, first_step, a.ctypes.data_as(C.POINTER(_U64)), len(a)), "tgp_replan_begin")

    def replan_wait(self):
        self._ck(lib().tgp_replan_wait(self._h), "tgp_replan_wait")

    def replan_commit(self):
        self._ck(lib().tgp_replan_commit(self._h), "tgp_replan_commit")

    def set_replan_keep(self, keep):
        self._ck(lib().tgp_set_replan_keep(self._h, int(keep)), "tgp_set_replan_keep")

    def set_budget(self, nbytes):
        self._ck(lib().tgp_set_budget(self._h, nbytes), "tgp_set_budget")

    def set_variant(self, variant, bits):
        self._ck(lib().tgp_set_variant(self._h, variant, bits), "tgp_set_variant")

    def set_object_bytes(self, nbytes):
        """Segment size of VAR_MANAGED_OBJECT, the object-level prefetcher."""
        self._ck(lib().tgp_set_object_bytes(self._h, nbytes), "tgp_set_object_bytes")

    def set_measured_times(self, op_ns):
        """Per-op kernel times in integer ns (0 = keep the analytic class); None or empty clears the log."""
        if op_ns is None or len(op_ns) == 0:
            self._ck(lib().tgp_set_measured_times(self._h, None, 0), "tgp_set_measured_times")
            return
        a = np.ascontiguousarray(op_ns, dtype=np.uint64)
        self._ck(lib().tgp_set_measured_times(self._h, a.ctypes.data_as(C.POINTER(_U64)), len(a)), "tgp_set_measured_times")

    def plan(self):
        self._ck(lib().tgp_plan(self._h), "tgp_plan")

    def plan_export(self, what):
        n = _U64()
        self._ck(lib().tgp_plan_export(self._h, what, None, C.byref(n)), "tgp_plan_export")
        buf = C.create_string_buffer(max(1, n.value))
        self._ck(lib().tgp_plan_export(self._h, what, buf, C.byref(n)), "tgp_plan_export")
        return buf.raw[:n.value]

    def plan_blobs(self, tail=False):
        """The plan in use as canonical blobs; tail=True: the tail plan that waits for replan_commit()."""
        f = X_TAIL if tail else 0
        return {k: self.plan_export(w | f) for k, w in (("classes", X_CLASSES), ("tensors", X_TENSORS), ("pins", X_PINS),
                                                        ("commands", X_COMMANDS), ("totals", X_TOTALS))}

    def set_arena(self, arena, nbytes):
        self._ck(lib().tgp_set_arena(self._h, _ptr(arena), nbytes), "tgp_set_arena")
        self._keep.append(arena)

    def model_bind(self, cfg: ModelCfg, roles, router_bias=None, workspace=None, ws_bytes=0, max_tokens=0):
        arr = (RoleEntry * len(roles))(*[RoleEntry(*r) for r in roles])
        rb = None if router_bias is None else np.ascontiguousarray(router_bias, dtype=np.float32)
        self._ck(lib().tgp_model_bind(self._h, C.byref(cfg), arr, len(roles), _ptr(rb), _ptr(workspace), ws_bytes, max_tokens), "tgp_model_bind")
        self._keep.append(workspace)

    def run_reset(self):
        self._ck(lib().tgp_run_reset(self._h), "tgp_run_reset")

    def step(self, kind, tokens_host, B, q_len, logits, argmax, compute_stream, copy_stream, want_stats=False):
        st = StepStats() if want_stats else None
        self._ck(lib().tgp_step(self._h, kind, _ptr(tokens_host), B, q_len, _ptr(logits), _ptr(argmax), _ptr(compute_stream),
                                _ptr(copy_stream), C.byref(st) if st is not None else None), "tgp_step")
        return st


    def expert_counts(self, L, E):
        """uint32 [steps run, L, E]: tokens routed to each expert since the last run_reset()."""
        n = _U64()
        self._ck(lib().tgp_expert_counts(self._h, None, C.byref(n)), "tgp_expert_counts")
        a = np.zeros(max(1, n.value), dtype=np.uint32)
        self._ck(lib().tgp_expert_counts(self._h, a.ctypes.data_as(C.POINTER(_U32)), C.byref(n)), "tgp_expert_counts")
        return a[:n.value].reshape(-1, L, E)

    def run_capture_begin(self, compute_stream, copy_stream):
        self._ck(lib().tgp_run_capture_begin(self._h, _ptr(compute_stream), _ptr(copy_stream)), "tgp_run_capture_begin")

    def run_capture_end(self):
        self._ck(lib().tgp_run_capture_end(self._h), "tgp_run_capture_end")

    def run_graph_launch(self, stream):
        self._ck(lib().tgp_run_graph_launch(self._h, _ptr(stream)), "tgp_run_graph_launch")

    def set_tap(self, tap, nbytes):
        self._ck(lib().tgp_set_tap(self._h, _ptr(tap), nbytes), "tgp_set_tap")
        self._keep.append(tap)

    def tap_index(self):
        """uint64 [records, 5]: op index, tag, sub-index, offset, bytes."""
        n = _U64()
        self._ck(lib().tgp_tap_index(self._h, None, C.byref(n)), "tgp_tap_index")
        a = np.zeros(max(1, n.value), dtype=np.uint64)
        self._ck(lib().tgp_tap_index(self._h, a.ctypes.data_as(C.POINTER(_U64)), C.byref(n)), "tgp_tap_index")
        return a[:n.value].reshape(-1, 5)

    def set_op_timing(self, enable):
        self._ck(lib().tgp_set_op_timing(self._h, int(enable)), "tgp_set_op_timing")

    def op_times(self):
        """(first op index, per-op milliseconds) of the last step that ran with op timing on."""
        first, n = _U32(), _U32()
        self._ck(lib().tgp_op_times(self._h, None, 0, C.byref(first), C.byref(n)), "tgp_op_times")
        ms = (C.c_float * max(1, n.value))()
        self._ck(lib().tgp_op_times(self._h, ms, n.value, C.byref(first), C.byref(n)), "tgp_op_times")
        return first.value, np.frombuffer(ms, dtype=np.float32, count=n.value).copy()


def managed_alloc(nbytes: int) -> int:
    p = _P()
    _k(lib().tgp_managed_alloc(C.byref(p), nbytes), "tgp_managed_alloc")
    return p.value


def managed_free(ptr: int):
    _k(lib().tgp_managed_free(ptr), "tgp_managed_free")


def managed_evict(ptr: int, nbytes: int):
    _k(lib().tgp_managed_evict(ptr, nbytes), "tgp_managed_evict")


def model_workspace_bytes(cfg: ModelCfg, max_tokens: int) -> int:
    n = _U64()
    rc = lib().tgp_model_workspace_bytes(C.byref(cfg), max_tokens, C.byref(n))
    if rc:
        raise TgpError(rc, "tgp_model_workspace_bytes")
    return n.value


def _tile_arrays(k_tiles, v_tiles):
    n = len(k_tiles)
    return (_P * max(1, n))(*[_ptr(t) for t in k_tiles]), (_P * max(1, n))(*[_ptr(t) for t in v_tiles]), n


def _k(rc, where):
    if rc:
        raise TgpError(rc, where)


def k_embed(table, tok, x, M, d, V, stream=None):
    _k(lib().tgp_k_embed(_ptr(table), _ptr(tok), _ptr(x), M, d, V, _ptr(stream)), "tgp_k_embed")


def k_embed_status():
    """(bad, row, token) of the first out-of-vocabulary token an embedding gather met, bad == 0 if none."""
    b, r, t = C.c_int(), _U32(), C.c_int32()
    _k(lib().tgp_k_embed_status(C.byref(b), C.byref(r), C.byref(t)), "tgp_k_embed_status")
    return b.value, r.value, t.value


def k_wait_test(limit_ns, withhold_step):
    _k(lib().tgp_k_wait_test(limit_ns, withhold_step), "tgp_k_wait_test")


def k_status_clear():
    _k(lib().tgp_k_status_clear(), "tgp_k_status_clear")


def k_rmsnorm(x, ldx, g, h, M, d, eps, stream=None):
    _k(lib().tgp_k_rmsnorm(_ptr(x), ldx, _ptr(g), _ptr(h), M, d, eps, _ptr(stream)), "tgp_k_rmsnorm")


def k_gemm(A, W, Cout, M, n, K, ldc, col0, accumulate, stream=None):
    _k(lib().tgp_k_gemm(_ptr(A), _ptr(W), _ptr(Cout), M, n, K, ldc, col0, int(accumulate), _ptr(stream)), "tgp_k_gemm")


def k_gemm_group(A, Ws, Couts, M, ns, K, ldcs, accumulate=False, stream=None):
    """Products of the same activations A [M, K] with several weight blocks Ws[s] [ns[s], K] into Couts[s] (row stride ldcs[s])."""
    c = len(Ws)
    _k(lib().tgp_k_gemm_group(_ptr(A), c, (_P * c)(*[_ptr(w) for w in Ws]), (_P * c)(*[_ptr(o) for o in Couts]),
                              (_U32 * c)(*ns), (_U32 * c)(*ldcs), M, K, int(accumulate), _ptr(stream)), "tgp_k_gemm_group")


def k_gemm_group_key(M, n, K):
    """Blocks with the same non-zero key may share a launch (0: launched alone)."""
    key = _U32(0)
    _k(lib().tgp_k_gemm_group_key(M, n, K, C.byref(key)), "tgp_k_gemm_group_key")
    return key.value


def k_gemm_group_select(enable):
    _k(lib().tgp_k_gemm_group_select(int(enable)), "tgp_k_gemm_group_select")


def k_gemm_select(impl):
    _k(lib().tgp_k_gemm_select(impl), "tgp_k_gemm_select")


def k_skinny_select(impl):
    _k(lib().tgp_k_skinny_select(impl), "tgp_k_skinny_select")


def k_gemv_overlap(enable):
    _k(lib().tgp_k_gemv_overlap(int(enable)), "tgp_k_gemv_overlap")


def k_gemm_chain(enable):
    _k(lib().tgp_k_gemm_chain(int(enable)), "tgp_k_gemm_chain")


def k_attn_select(impl):
    _k(lib().tgp_k_attn_select(impl), "tgp_k_attn_select")


def k_gemm_tc_variant(v):
    _k(lib().tgp_k_gemm_tc_variant(v), "tgp_k_gemm_tc_variant")


def k_gemm_last_kernel():
    buf = C.create_string_buffer(96)
    _k(lib().tgp_k_gemm_last_kernel(buf, 96), "tgp_k_gemm_last_kernel")
    return buf.value.decode()


def k_attn_decode_select(impl):
    _k(lib().tgp_k_attn_decode_select(impl), "tgp_k_attn_decode_select")


def k_swiglu_epilogue(enable):
    _k(lib().tgp_k_swiglu_epilogue(int(enable)), "tgp_k_swiglu_epilogue")


def k_merge_copies(enable):
    _k(lib().tgp_k_merge_copies(int(enable)), "tgp_k_merge_copies")


def k_decode_fuse(enable):
    _k(lib().tgp_k_decode_fuse(int(enable)), "tgp_k_decode_fuse")


def k_attn_status():
    e = C.c_int()
    _k(lib().tgp_k_attn_status(C.byref(e)), "tgp_k_attn_status")
    return e.value


def k_gemm_status():
    e = C.c_int()
    _k(lib().tgp_k_gemm_status(C.byref(e)), "tgp_k_gemm_status")
    return e.value


def k_rope_tables(Dh, max_len, base, cos, sin):
    _k(lib().tgp_k_rope_tables(Dh, max_len, base, _ptr(cos), _ptr(sin)), "tgp_k_rope_tables")


def k_rope_kv(q32, k32, v32, qb, k_tiles, v_tiles, cos, sin, cfg, B, q_len, pos0, stream=None):
    ka, va, n = _tile_arrays(k_tiles, v_tiles)
    _k(lib().tgp_k_rope_kv(_ptr(q32), _ptr(k32), _ptr(v32), _ptr(qb), ka, va, n, _ptr(cos), _ptr(sin), C.byref(cfg), B, q_len, pos0, _ptr(stream)), "tgp_k_rope_kv")


def k_attn(qb, k_tiles, v_tiles, ob, cfg, B, q_len, pos0, scratch=None, stream=None):
    ka, va, n = _tile_arrays(k_tiles, v_tiles)
    _k(lib().tgp_k_attn(_ptr(qb), ka, va, n, _ptr(ob), C.byref(cfg), B, q_len, pos0, _ptr(scratch), _ptr(stream)), "tgp_k_attn")


STATIC_SCRATCH_BYTES = 4 << 20


def k_attn_decode_static(qb, k_tiles, v_tiles, ob, cfg, B, pos0, stream=None):
    """Decode attention whose scratch is a fixed array inside the library: for callers that cannot allocate
    device memory.  Raises TgpError(E_TOO_LARGE) when the partials would not fit in STATIC_SCRATCH_BYTES."""
    ka, va, n = _tile_arrays(k_tiles, v_tiles)
    _k(lib().tgp_k_attn_decode_static(_ptr(qb), ka, va, n, _ptr(ob), C.byref(cfg), B, pos0, _ptr(stream)), "tgp_k_attn_decode_static")


def k_attn_scratch_bytes(cfg):
    n = _U64()
    _k(lib().tgp_k_attn_scratch_bytes(C.byref(cfg), C.byref(n)), "tgp_k_attn_scratch_bytes")
    return n.value


def k_swiglu(g, u, ab, n, stream=None):
    _k(lib().tgp_k_swiglu(_ptr(g), _ptr(u), _ptr(ab), n, _ptr(stream)), "tgp_k_swiglu")


def k_argmax(logits, out, B, V, stream=None):
    _k(lib().tgp_k_argmax(_ptr(logits), _ptr(out), B, V, _ptr(stream)), "tgp_k_argmax")
