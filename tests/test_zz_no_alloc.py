"""The allocation-free decode-attention entry point against the ordinary one.

Some users of this library run where they cannot allocate device memory: the device budget is already
spent on the arena and workspace, or an allocation's implicit synchronisation would stall their serving
loop.  For them tgp_k_attn_decode_static() keeps its scratch in a fixed array inside the library.  Here it
is called through the C ABI twice in a row (the array is shared and keeps the previous call's contents) and
must give what tgp_k_attn() gives with caller scratch, and what the CPU oracle's attention gives on the same
queries and cache (the rule the kernel tests use: within one bf16 ulp of the largest output).  This file sorts last on purpose: a run that stops at
the first failure has then already run everything else.
"""
import numpy as np
import pytest

import seeded_inputs as si

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.forward import OracleModel, bf16_round  # noqa: E402
from paper_2609_06172_b200 import binding as tb  # noqa: E402
from paper_2609_06172_b200.session import model_cfg  # noqa: E402

DEV = "cuda:0"


def _case(cfg, B, pos0, seed):
    nt = cfg.n_tiles
    n = B * cfg.Hkv * cfg.TK * cfg.Dh
    kt = [torch.from_numpy(si.normal_bf16_bits(seed, 100 + j, 0, n).view(np.int16)).to(DEV).view(torch.bfloat16) * 40 for j in range(nt)]
    vt = [torch.from_numpy(si.normal_bf16_bits(seed, 200 + j, 0, n).view(np.int16)).to(DEV).view(torch.bfloat16) * 40 for j in range(nt)]
    qb = torch.from_numpy(si.normal_bf16_bits(seed, 7, 0, B * cfg.Hq * cfg.Dh).view(np.int16)).to(DEV).view(torch.bfloat16) * 40
    return kt, vt, qb


@pytest.mark.parametrize("shape", [dict(Hq=32, Hkv=8, Dh=64, TK=128, B=1, S=512, T=128), dict(Hq=8, Hkv=2, Dh=128, TK=16, B=3, S=40, T=9)])
def test_static_scratch_variant_matches_caller_scratch_variant_twice_in_a_row(shape):
    cfg = si.ModelConfig("na", L=1, d=shape["Hq"] * shape["Dh"], F=64, V=64, seed=3, budget_rule="half_w", **shape)
    mc = model_cfg(cfg)
    scratch = torch.empty(tb.k_attn_scratch_bytes(mc) // 4, dtype=torch.float32, device=DEV)
    for call, pos0 in enumerate((cfg.max_len - 1, cfg.S // 2)):          # second call: fewer tiles, stale partials left behind
        kt, vt, qb = _case(cfg, cfg.B, pos0, seed=11 + call)
        want = torch.empty(cfg.B, cfg.Hq * cfg.Dh, dtype=torch.bfloat16, device=DEV)
        got = torch.full_like(want, float("nan"))
        tb.k_attn(qb, kt, vt, want, mc, cfg.B, 1, pos0, scratch)
        tb.k_attn_decode_static(qb, kt, vt, got, mc, cfg.B, pos0)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        # same kernels, same inputs: bf16 outputs within one ulp (the tolerance the kernel tests use); in fact equal
        g, w = got.float().cpu().numpy(), want.float().cpu().numpy()
        assert (np.abs(g - w) <= np.abs(w) * 2.0 ** -7).all()
        assert np.array_equal(g, w)
        # and against the oracle: softmax(q K^T / sqrt(Dh)) V over the pos0 + 1 cached keys, from the same bf16 inputs
        om = OracleModel(cfg, {})
        cache = lambda tiles: torch.stack([x.view(cfg.B, cfg.Hkv, cfg.TK, cfg.Dh) for x in tiles], dim=2).reshape(cfg.B, cfg.Hkv, -1, cfg.Dh).float().cpu().numpy()
        om.K[0], om.V[0] = cache(kt)[:, :, :cfg.max_len], cache(vt)[:, :, :cfg.max_len]
        att = om.attention(0, qb.float().cpu().numpy().reshape(cfg.B, 1, cfg.Hq, cfg.Dh), pos0).reshape(cfg.B, cfg.Hq * cfg.Dh)
        assert np.abs(g - att).max() < 2.0 ** -7 * np.abs(att).max() + 1e-6
        assert np.mean(np.abs(g - bf16_round(att))) < 3e-3 * np.abs(att).mean()


def test_static_scratch_variant_rejects_sizes_beyond_its_fixed_array():
    cfg = si.ModelConfig("big", L=1, d=8192, Hq=64, Hkv=8, Dh=128, F=64, V=64, B=16, S=2048, T=64, TK=64, seed=3, budget_rule="half_w")
    mc = model_cfg(cfg)
    assert cfg.B * cfg.Hq * cfg.n_tiles * (cfg.Dh + 2) * 4 > tb.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(16, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(tb.TgpError) as ei:
        tb.k_attn_decode_static(dummy, [dummy] * cfg.n_tiles, [dummy] * cfg.n_tiles, dummy, mc, cfg.B, 100)
    assert ei.value.code == tb.E_TOO_LARGE
    torch.cuda.synchronize()
