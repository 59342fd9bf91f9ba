"""The synthetic workload: sizes match the five configurations, the generator is deterministic and ~N(0, 0.02)."""
import numpy as np
import pytest

import seeded_inputs as si

# (weight bytes, KV bytes, budget) derived by hand from the shapes of the five configurations
EXPECTED = {
    1: (12_587_520, 196_608, 6_392_064),
    2: (2_208_436_224, 20_971_520, 1_104_218_112),
    3: (16_060_522_496, 1_342_177_280, 8 << 30),
    4: (141_107_412_992, 11_072_962_560, 64 << 30),
    5: (93_405_585_408, 2_684_354_560, 40 << 30),
}


@pytest.mark.parametrize("c", [1, 2, 3, 4, 5])
def test_layout_sizes(c):
    lay = si.build_layout(si.CONFIGS[c])
    assert (lay.weight_bytes, lay.kv_bytes, lay.budget) == EXPECTED[c]
    # sub-ranges are disjoint, aligned and inside the pool
    end = 0
    for t in lay.tensors:
        assert t.pool_off % si.POOL_ALIGN == 0 and t.pool_off >= end
        end = t.pool_off + t.size
        assert t.size <= max(lay.sub_range_cap, t.cols * 2) or t.kind in (si.K_EMBED, si.K_KT, si.K_VT, si.K_ROUTER)
    assert end <= lay.pool_bytes
    assert sum(t.size for t in lay.tensors if t.kind < si.K_KT) == lay.weight_bytes


def test_sub_range_cap_rule():
    assert si.sub_range_cap(6_392_064) == 512 << 10
    assert si.sub_range_cap(1 << 20) == 128 << 10
    assert si.sub_range_cap(1_104_218_112) == 32 << 20
    assert si.sub_range_cap(64 << 30) == 32 << 20


def test_generator_statistics_and_determinism():
    a = si.normal_bf16_bits(123, 7, 0, 1 << 20)
    b = si.normal_bf16_bits(123, 7, 0, 1 << 20, threads=2)
    assert np.array_equal(a, b)
    x = si.bf16_bits_to_f32(a).astype(np.float64)
    assert abs(x.mean()) < 2e-4
    assert abs(x.std() - 0.02) < 0.02 * 0.01
    # a block generated at an offset equals the same elements of the whole stream
    c = si.normal_bf16_bits(123, 7, 1000, 5000)
    assert np.array_equal(c, a[1000:6000])
    # different roles differ
    assert not np.array_equal(a[:64], si.normal_bf16_bits(123, 8, 0, 64))


def test_bf16_rounding_matches_torch():
    import torch
    rng = np.random.default_rng(0)
    x = rng.standard_normal(100000).astype(np.float32)
    x[:4] = np.array([1.00390625, 1.01171875, -1.00390625, 3.0], dtype=np.float32)      # exact ties and an exact value
    ours = si.bf16_bits_to_f32(si.f32_to_bf16_bits(x))
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours, ref)


def test_prompt_range_and_determinism():
    cfg = si.CONFIGS[2]
    t = si.prompt_tokens(cfg)
    assert t.shape == (cfg.B, cfg.S) and t.min() >= 0 and t.max() < cfg.V
    assert np.array_equal(t, si.prompt_tokens(cfg))
    assert len(np.unique(t)) > cfg.S // 2


def test_router_bias_is_zipf_permutation():
    cfg = si.CONFIGS[5]
    b = si.router_bias(cfg)
    assert b.shape == (cfg.L, cfg.E)
    p = np.exp(b.astype(np.float64))
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-5)
    ref = np.array([r ** -1.2 for r in range(1, 9)]); ref /= ref.sum()
    for l in range(cfg.L):
        assert np.allclose(np.sort(p[l])[::-1], ref, atol=1e-6)
    assert len({tuple(np.argsort(-b[l])) for l in range(cfg.L)}) > 1


def test_torch_generator_matches_numpy_generator_bit_for_bit():
    import torch
    cfg = si.CONFIGS[1]
    lay = si.build_layout(cfg)
    a = np.zeros(lay.pool_bytes, dtype=np.uint8)
    si.fill_pool(lay, a)
    b = torch.zeros(lay.pool_bytes, dtype=torch.uint8)
    si.fill_pool_torch(lay, b, device="cuda:0" if torch.cuda.is_available() else "cpu", chunk=100000)
    assert np.array_equal(a, b.numpy())
