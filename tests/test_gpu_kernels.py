"""Kernel parity on the GPU: every kernel of the path, called through the C ABI, against the CPU oracle
on the same seeded inputs; sizes span several tiles and ragged tails, plus the degenerate cases."""
from dataclasses import replace

import numpy as np
import pytest

import seeded_inputs as si

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.forward import OracleModel, bf16_round  # noqa: E402
from paper_2609_06172_b200 import binding as tb  # noqa: E402
from paper_2609_06172_b200.session import model_cfg  # noqa: E402

DEV = "cuda:0"
KCFG = si.ModelConfig("k", L=1, d=128, Hq=4, Hkv=2, Dh=64, F=256, V=512, B=2, S=8, T=8, TK=4, seed=7, budget_rule="half_w")


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).to(DEV).view(torch.bfloat16)


def rnd_bits(role, n):
    return si.normal_bf16_bits(1234, role, 0, n)


def oracle():
    lay = si.build_layout(KCFG)
    return OracleModel(KCFG, si.weights_as_bits(lay))


def bf16_close(got_f32, want_f32, frac=0.01):
    """Equal up to one bf16 ulp, and different at all in at most `frac` of the entries (rounding flips
    where fp32 summation order differs by a last bit)."""
    got, want = np.asarray(got_f32, np.float32), np.asarray(want_f32, np.float32)
    tol = np.maximum(np.abs(want), 1e-30) * 2.0 ** -7
    assert (np.abs(got - want) <= tol).all(), float(np.abs(got - want).max())
    assert (got != want).mean() <= frac


@pytest.mark.parametrize("M,n,K", [(1, 300, 256), (1, 4096, 2048), (2, 129, 64), (3, 1000, 512), (8, 1030, 512),
                                   (13, 77, 128), (16, 260, 1024), (17, 64, 96), (33, 130, 96), (200, 260, 1024),
                                   (64, 64, 32), (1, 1, 8), (70, 5, 8), (129, 257, 72), (300, 520, 1096), (512, 2048, 2048),
                                   (1000, 136, 8192),
                                   # few rows, long K at M <= 2: the split-K GEMV (two rows per CTA; one row per CTA up to 1024 rows),
                                   # odd row counts, K not a multiple of the 256-element chunk, more CTAs than resident slots
                                   (1, 2048, 8192), (2, 2051, 8200), (1, 513, 8192), (2, 1, 16384), (1, 4735, 8192),
                                   # 33 - 64 activation rows on a block of few rows: two weight-streaming launches of half the rows
                                   (33, 1030, 512), (48, 2049, 4096), (64, 130, 96), (40, 4090, 64),
                                   # ... and on blocks of many rows the tiled GEMM with the weights as its 128-row operand
                                   (40, 4720, 64), (64, 4096, 1032), (20, 8200, 128)])
@pytest.mark.parametrize("accumulate", [0, 1])
def test_gemm_matches_oracle(M, n, K, accumulate):
    a_bits, w_bits = rnd_bits(1, M * K).reshape(M, K), rnd_bits(2, n * K).reshape(n, K)
    A, W = bf16_dev(a_bits), bf16_dev(w_bits)
    ldc, col0 = n + 24, 8
    c0 = np.random.default_rng(M * n).standard_normal((M, ldc)).astype(np.float32) * 0.01
    Cd = torch.from_numpy(c0.copy()).to(DEV)
    tb.k_gemm(A, W, Cd, M, n, K, ldc, col0, accumulate)
    torch.cuda.synchronize()
    got = Cd.cpu().numpy()
    o = oracle()
    want = o.linear(si.bf16_bits_to_f32(a_bits), si.bf16_bits_to_f32(w_bits).astype(np.float64)).astype(np.float64)
    exp = c0.astype(np.float64).copy()
    exp[:, col0:col0 + n] = want + (c0[:, col0:col0 + n] if accumulate else 0)
    scale = np.abs(want).max() + 1e-6
    assert np.abs(got - exp).max() < 2e-5 * max(scale, 0.01) + 1e-7
    assert np.array_equal(got[:, :col0], c0[:, :col0]) and np.array_equal(got[:, col0 + n:], c0[:, col0 + n:])


def test_tensor_core_gemm_agrees_with_cuda_core_gemm_and_reports_no_timeout():
    """Same inputs through both M > 16 kernels: the tcgen05 path and the CUDA-core tiles (an on-device cross-check
    besides the oracle), then the tensor-core kernel's bounded-wait error word must still be zero."""
    M, n, K = 640, 1408, 2048
    A, W = bf16_dev(rnd_bits(5, M * K).reshape(M, K)), bf16_dev(rnd_bits(6, n * K).reshape(n, K))
    outs = []
    for impl in (0, 1):
        tb.k_gemm_select(impl)
        Cd = torch.zeros(M, n, dtype=torch.float32, device=DEV)
        tb.k_gemm(A, W, Cd, M, n, K, n, 0, 0)
        torch.cuda.synchronize()
        outs.append(Cd.cpu().numpy())
    tb.k_gemm_select(0)
    assert np.abs(outs[0] - outs[1]).max() < 2e-5 * np.abs(outs[1]).max()
    assert np.abs(outs[0]).max() > 0
    assert tb.k_gemm_status() == 0


@pytest.mark.parametrize("M,n,K,acc", [(300, 520, 1096, 0), (129, 257, 72, 1), (1024, 1536, 512, 0), (640, 2300, 2048, 1), (4096, 4096, 256, 0)])
def test_persistent_tensor_core_gemm_matches_per_tile_kernel_and_oracle(M, n, K, acc):
    """The paired 256x256 kernel and the persistent 128x256 kernel (forced, even on small problems: ragged tiles, a pair
    whose second CTA has no valid row, fewer tiles than SMs, several tiles per CTA) against the per-tile kernel and the
    oracle."""
    a_bits, w_bits = rnd_bits(11, M * K).reshape(M, K), rnd_bits(12, n * K).reshape(n, K)
    A, W = bf16_dev(a_bits), bf16_dev(w_bits)
    c0 = np.random.default_rng(7).standard_normal((M, n)).astype(np.float32) * 0.01
    outs = []
    for variant in (3, 2, 1):
        tb.k_gemm_tc_variant(variant)
        Cd = torch.from_numpy(c0.copy()).to(DEV)
        tb.k_gemm(A, W, Cd, M, n, K, n, 0, acc)
        torch.cuda.synchronize()
        outs.append(Cd.cpu().numpy())
    tb.k_gemm_tc_variant(0)
    assert tb.k_gemm_status() == 0
    want = oracle().linear(si.bf16_bits_to_f32(a_bits), si.bf16_bits_to_f32(w_bits).astype(np.float64)).astype(np.float64) + (c0 if acc else 0)
    scale = np.abs(want).max()
    for o in outs:
        assert np.abs(o - want).max() < 2e-5 * scale + 1e-7
    assert np.abs(outs[0] - outs[2]).max() < 2e-5 * scale + 1e-7 and np.abs(outs[1] - outs[2]).max() < 2e-5 * scale + 1e-7


@pytest.mark.parametrize("M,n,K,acc", [(17, 300, 264, 0), (32, 4100, 1024, 1), (33, 1030, 512, 1), (64, 130, 96, 0), (65, 2049, 1024, 1),
                                       (128, 4096, 512, 0), (100, 129, 72, 1), (48, 8200, 256, 0)])
def test_tensor_core_gemm_with_the_weights_as_the_128_row_operand(M, n, K, acc):
    """Up to 128 activation rows: the per-tile kernel with its operands swapped (tile rows are weight rows, the tile is
    stored transposed), forced, against the oracle; ragged weight tiles, ragged token counts, a column offset."""
    a_bits, w_bits = rnd_bits(13, M * K).reshape(M, K), rnd_bits(14, n * K).reshape(n, K)
    A, W = bf16_dev(a_bits), bf16_dev(w_bits)
    ldc, col0 = n + 12, 4
    c0 = np.random.default_rng(9).standard_normal((M, ldc)).astype(np.float32) * 0.01
    tb.k_gemm_tc_variant(4)
    tb.k_skinny_select(1)            # 17 - 32 rows reach the tiled GEMM only with the weight-streaming kernel switched off
    Cd = torch.from_numpy(c0.copy()).to(DEV)
    tb.k_gemm(A, W, Cd, M, n, K, ldc, col0, acc)
    torch.cuda.synchronize()
    tb.k_gemm_tc_variant(0)
    tb.k_skinny_select(0)
    assert tb.k_gemm_status() == 0
    got = Cd.cpu().numpy()
    want = oracle().linear(si.bf16_bits_to_f32(a_bits), si.bf16_bits_to_f32(w_bits).astype(np.float64)).astype(np.float64)
    exp = c0.astype(np.float64).copy()
    exp[:, col0:col0 + n] = want + (c0[:, col0:col0 + n] if acc else 0)
    assert np.abs(got - exp).max() < 2e-5 * max(np.abs(want).max(), 0.01) + 1e-7
    assert np.array_equal(got[:, :col0], c0[:, :col0]) and np.array_equal(got[:, col0 + n:], c0[:, col0 + n:])


# (M, K, n, residual): the weight-block products of the prefill steps the benchmark times - M = B * S of the 8B shape (8 x 1024),
# the MoE shape (32 x 512) and the 70B shape (16 x 2048); K = d or FFN; n = rows of one 32 MiB sub-range block of that matrix
REAL_PREFILL = [(8192, 4096, 4096, 0), (8192, 14336, 1152, 1), (16384, 4096, 4096, 0), (32768, 8192, 2048, 0), (32768, 28672, 512, 1)]


@pytest.mark.parametrize("M,K,n,acc", REAL_PREFILL)
def test_gemm_at_the_real_prefill_shapes_sampled_rows_against_the_oracle(M, K, n, acc):
    """Full-size prefill products in the launch configuration the benchmark times (automatic kernel choice: the paired
    tcgen05 kernel).  A full CPU product would take minutes, and an output row depends on one activation row only, so
    the oracle recomputes 64 sampled rows - first, last, the rows around every 128- and 256-row tile edge it can hit,
    and seeded random ones - from the same bf16 inputs, in double.  The rows in between are covered by a checksum
    property that holds at any size: the column sums of C equal (column sums of A) . W^T."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(M * 31 + K)
    A = torch.randn((M, K), device=DEV, generator=gen).bfloat16()
    W = (torch.randn((n, K), device=DEV, generator=gen) * 0.02).bfloat16()
    c0 = (torch.randn((M, n), device=DEV, generator=gen) * 0.5).float() if acc else None
    Cd = c0.clone() if acc else torch.empty((M, n), dtype=torch.float32, device=DEV)
    tb.k_gemm(A, W, Cd, M, n, K, n, 0, acc)
    torch.cuda.synchronize()
    assert tb.k_gemm_status() == 0
    rng = np.random.default_rng(M + K)
    rows = sorted(set([0, 1, 127, 128, 255, 256, M // 2 - 1, M // 2, M - 257, M - 256, M - 129, M - 128, M - 2, M - 1] + rng.integers(0, M, 50).tolist()))[:64]
    ridx = torch.tensor(rows, device=DEV)
    a_rows = si.bf16_bits_to_f32(A[ridx].view(torch.int16).cpu().numpy().view(np.uint16))
    w_bits = W.view(torch.int16).cpu().numpy().view(np.uint16)
    want = oracle().linear(a_rows, si.bf16_bits_to_f32(w_bits).astype(np.float64)).astype(np.float64)
    if acc:
        want = want + c0[ridx].cpu().numpy().astype(np.float64)
    got = Cd[ridx].cpu().numpy().astype(np.float64)
    scale = np.abs(want).max()
    # 2e-5 of the largest output holds up to K = 8192 (every other GEMM test).  The tensor cores add each 16-deep partial
    # product into the fp32 accumulator without round-to-nearest, so the error has a part that grows linearly with the
    # K / 16 accumulation steps (bound: K / 16 * 2^-23 = 2.1e-4 at K = 28672; measured 3.2e-5): the tolerance grows with K
    tol = 2e-5 * max(1.0, K / 8192)
    assert np.abs(got - want).max() < tol * scale + 1e-7, (np.abs(got - want).max(), scale)
    # every row, through a property: sum_m C[m, j] = (sum_m A[m, :]) . W[j, :]  (+ sum_m C0[m, j]), in double
    colsum = Cd.double().sum(dim=0).cpu().numpy()
    asum = A.double().sum(dim=0).cpu().numpy()
    ref = si.bf16_bits_to_f32(w_bits).astype(np.float64) @ asum + (c0.double().sum(dim=0).cpu().numpy() if acc else 0.0)
    # fp32 accumulation error of one output element is ~1e-6 of its scale; M of them add up at random
    # (the accumulator's rounding bias has one sign per column, so over M rows it adds up linearly in the worst case)
    assert np.abs(colsum - ref).max() < tol * scale * M * 0.25 + 1e-6, (np.abs(colsum - ref).max(), scale)
    # and no element is non-finite or left unwritten
    assert bool(torch.isfinite(Cd).all())


@pytest.mark.parametrize("variant,M,n,K", [(1, 256, 256, 512), (2, 384, 512, 512), (3, 512, 512, 1024)])
def test_tensor_core_gemm_gives_up_on_a_wait_that_runs_out_and_recovers(variant, M, n, K):
    """Failure detection without a fault: with the wait limit set to 2 ms and the TMA thread of the first CTA (pair)
    leaving out its second load step, the MMA thread's wait for that stage runs out.  The kernel must return by itself,
    the error word must name the wait (role 2 = MMA issuer), the CTA that gave up must have stored nothing, every other
    CTA's tile must be right, and - limits restored, error word cleared - the next launch must be correct again."""
    a_bits, w_bits = rnd_bits(51, M * K).reshape(M, K), rnd_bits(52, n * K).reshape(n, K)
    A, W = bf16_dev(a_bits), bf16_dev(w_bits)
    want = oracle().linear(si.bf16_bits_to_f32(a_bits), si.bf16_bits_to_f32(w_bits).astype(np.float64)).astype(np.float64)
    SENT = 12345.0
    tb.k_status_clear()
    tb.k_gemm_tc_variant(variant)
    try:
        tb.k_wait_test(2_000_000, 1)
        Cd = torch.full((M, n), SENT, dtype=torch.float32, device=DEV)
        tb.k_gemm(A, W, Cd, M, n, K, n, 0, 0)
        torch.cuda.synchronize()                              # returns: nothing hangs, nothing faults
        code = tb.k_gemm_status()
        assert code >> 8 == 2, hex(code)                      # the MMA issuer's wait for a stage ran out first
        got = Cd.cpu().numpy()
        untouched = got == SENT
        rows, cols = (256, 256) if variant == 3 else (128, 256 if variant == 2 else 128)
        assert untouched[:rows, :cols].all()                  # the first CTA (pair) owns the first tile: nothing stored
        done = ~untouched
        assert done.sum() == M * n - rows * cols              # every other tile was stored, and correctly
        assert np.abs(got[done] - want[done]).max() < 2e-5 * np.abs(want).max() + 1e-7
    finally:
        tb.k_wait_test(0, -1)
        tb.k_status_clear()
    Cd = torch.zeros((M, n), dtype=torch.float32, device=DEV)
    tb.k_gemm(A, W, Cd, M, n, K, n, 0, 0)
    torch.cuda.synchronize()
    tb.k_gemm_tc_variant(0)
    assert tb.k_gemm_status() == 0
    assert np.abs(Cd.cpu().numpy() - want).max() < 2e-5 * np.abs(want).max() + 1e-7


@pytest.mark.parametrize("Dh", [64, 128])
def test_tensor_core_attention_gives_up_on_a_wait_that_runs_out_and_recovers(Dh):
    """The same for the tcgen05 attention kernel: the first CTA's TMA thread never requests its second V block, the
    roles that depend on it - the P V issuer (code 3: a K/V load), the softmax warps (1: S, 2: P V), the S issuer - all
    start waiting within microseconds of each other and the first whose 2 ms run out records its code; that CTA stores
    nothing, the others finish, and the next launch is correct."""
    cfg = replace(KCFG, Dh=Dh, Hq=4, Hkv=2, TK=64, S=256, T=0, B=2, d=4 * Dh)
    mc = model_cfg(cfg)
    B, S = cfg.B, cfg.S
    kt, vt = make_tiles(cfg, B)
    for j, (k, v) in enumerate(zip(kt, vt)):
        k.copy_(bf16_dev(rnd_bits(60 + j, k.numel())) * 30)
        v.copy_(bf16_dev(rnd_bits(70 + j, v.numel())) * 30)
    qb = (bf16_dev(rnd_bits(80, B * S * cfg.Hq * Dh)) * 30).view(B * S, cfg.Hq * Dh)
    o = OracleModel(cfg, {})
    o.K[0], o.V[0] = tiles_to_cache(kt, cfg, B)[:, :, :S], tiles_to_cache(vt, cfg, B)[:, :, :S]
    want = o.attention(0, qb.float().cpu().numpy().reshape(B, S, cfg.Hq, Dh), 0)
    tb.k_status_clear()
    tb.k_attn_select(3)
    try:
        tb.k_wait_test(2_000_000, 1)
        ob = torch.full((B * S, cfg.Hq * Dh), 768.0, dtype=torch.bfloat16, device=DEV)
        tb.k_attn(qb, kt, vt, ob, mc, B, S, 0, None)
        torch.cuda.synchronize()
        assert tb.k_attn_status() in (1, 2, 3)
        got = ob.float().cpu().numpy().reshape(B, S, cfg.Hq, Dh)
        untouched = got == 768.0
        # the grid's first CTA is the last query block (longest first) of head 0, sequence 0
        assert untouched[0, 128:, 0].all() and untouched.sum() == 128 * Dh
        done = ~untouched
        assert np.abs(got[done] - want[done]).max() < 2.0 ** -7 * np.abs(want).max() + 1e-6
    finally:
        tb.k_wait_test(0, -1)
        tb.k_status_clear()
    ob = torch.zeros((B * S, cfg.Hq * Dh), dtype=torch.bfloat16, device=DEV)
    tb.k_attn(qb, kt, vt, ob, mc, B, S, 0, None)
    torch.cuda.synchronize()
    tb.k_attn_select(0)
    assert tb.k_attn_status() == 0
    assert np.abs(ob.float().cpu().numpy().reshape(B, S, cfg.Hq, Dh) - want).max() < 2.0 ** -7 * np.abs(want).max() + 1e-6


def test_gemm_rejects_bad_arguments_and_accepts_empty():
    A = torch.zeros(8, 16, dtype=torch.bfloat16, device=DEV)
    Cd = torch.zeros(8, 8, dtype=torch.float32, device=DEV)
    with pytest.raises(tb.TgpError):
        tb.k_gemm(A, A, Cd, 8, 8, 12, 8, 0, 0)          # K % 8
    with pytest.raises(tb.TgpError):
        tb.k_gemm(A, A, Cd, 8, 8, 16, 8, 4, 0)          # col0 + n > ldc
    tb.k_gemm(A, A, Cd, 0, 8, 16, 8, 0, 0)              # empty M: no launch, no error
    torch.cuda.synchronize()


@pytest.mark.parametrize("M,d", [(1, 128), (5, 256), (37, 2048), (3, 8192)])
def test_rmsnorm_and_embed(M, d):
    V = 300
    tab_bits = rnd_bits(3, V * d).reshape(V, d)
    tok = (np.arange(M, dtype=np.int32) * 37 + 5) % V
    x = torch.empty(M, d, dtype=torch.float32, device=DEV)
    tb.k_embed(bf16_dev(tab_bits), torch.from_numpy(tok).to(DEV), x, M, d, V)
    torch.cuda.synchronize()
    assert np.array_equal(x.cpu().numpy(), si.bf16_bits_to_f32(tab_bits)[tok])
    assert tb.k_embed_status()[0] == 0
    xin = (np.random.default_rng(d).standard_normal((M, d)) * 3).astype(np.float32)
    g_bits = si.f32_to_bf16_bits(1.0 + 0.1 * np.random.default_rng(1).standard_normal(d).astype(np.float32))
    h = torch.empty(M, d, dtype=torch.bfloat16, device=DEV)
    tb.k_rmsnorm(torch.from_numpy(xin).to(DEV), d, bf16_dev(g_bits), h, M, d, 1e-5)
    torch.cuda.synchronize()
    o = oracle()
    want = o.rmsnorm(xin, si.bf16_bits_to_f32(g_bits).astype(np.float64))
    bf16_close(h.float().cpu().numpy(), want)


def test_embed_zeroes_rows_of_tokens_outside_the_vocabulary_and_records_the_first():
    """A token id outside [0, V) must never index the table (in an oversubscribed run the table may be mapped host
    memory): its row is zeros, the others are gathered as usual, and the error word names the row and the id."""
    V, d, M = 50, 64, 6
    tab_bits = rnd_bits(11, V * d).reshape(V, d)
    tok = np.array([3, V, 7, -1, 49, 2 ** 31 - 1], dtype=np.int32)
    x = torch.full((M, d), 7.0, dtype=torch.float32, device=DEV)
    tb.k_status_clear()
    tb.k_embed(bf16_dev(tab_bits), torch.from_numpy(tok).to(DEV), x, M, d, V)
    torch.cuda.synchronize()
    got = x.cpu().numpy()
    ok = (tok >= 0) & (tok < V)
    assert np.array_equal(got[ok], si.bf16_bits_to_f32(tab_bits)[tok[ok]])
    assert not got[~ok].any()
    bad, row, token = tb.k_embed_status()
    assert bad == 1 and row in (1, 3, 5) and token == int(tok[row])
    tb.k_status_clear()
    assert tb.k_embed_status()[0] == 0


def test_argmax_of_a_row_of_nans_is_a_legal_token():
    V = 5000
    lg = np.full((3, V), np.nan, dtype=np.float32)
    lg[1] = -np.inf
    lg[2, 4000] = 1.0
    am = torch.full((3,), -7, dtype=torch.int32, device=DEV)
    tb.k_argmax(torch.from_numpy(lg).to(DEV), am, 3, V)
    torch.cuda.synchronize()
    got = am.cpu().numpy()
    assert got[0] == 0 and got[1] == 0 and 0 <= got[2] < V


def make_tiles(cfg, B):
    nt = cfg.n_tiles
    k = [torch.zeros(B * cfg.Hkv * cfg.TK * cfg.Dh, dtype=torch.bfloat16, device=DEV) for _ in range(nt)]
    v = [torch.zeros(B * cfg.Hkv * cfg.TK * cfg.Dh, dtype=torch.bfloat16, device=DEV) for _ in range(nt)]
    return k, v


def tiles_to_cache(tiles, cfg, B):
    """[n_tiles] x [B, Hkv, TK, Dh] -> [B, Hkv, n_tiles*TK, Dh] fp32"""
    t = torch.stack([x.view(B, cfg.Hkv, cfg.TK, cfg.Dh) for x in tiles], dim=2)
    return t.reshape(B, cfg.Hkv, -1, cfg.Dh).float().cpu().numpy()


@pytest.mark.parametrize("attn_impl", [3, 2])
@pytest.mark.parametrize("Dh,Hq,Hkv,TK,S,T", [(64, 4, 2, 4, 9, 7), (128, 8, 2, 16, 40, 5), (64, 4, 4, 8, 33, 3), (128, 8, 1, 64, 130, 2),
                                             (64, 6, 2, 32, 70, 3)])      # three query heads per KV head: the per-head decode kernel
def test_rope_kv_and_attention_prefill_then_decode(Dh, Hq, Hkv, TK, S, T, attn_impl):
    B = 2
    tb.k_attn_select(attn_impl)
    cfg = replace(KCFG, Dh=Dh, Hq=Hq, Hkv=Hkv, TK=TK, S=S, T=T, B=B, d=Hq * Dh)
    lay_w = {(k, 0, -1): rnd_bits(k, 8).reshape(1, 8) for k in range(13)}
    o = OracleModel(cfg, lay_w)
    mc = model_cfg(cfg)
    cos = torch.empty(cfg.max_len * Dh // 2, dtype=torch.float32, device=DEV)
    sin = torch.empty_like(cos)
    tb.k_rope_tables(Dh, cfg.max_len, cfg.rope_base, cos, sin)
    assert np.array_equal(cos.cpu().numpy().reshape(cfg.max_len, Dh // 2), o.cos)
    kt, vt = make_tiles(cfg, B)
    scratch = torch.empty(tb.k_attn_scratch_bytes(mc) // 4, dtype=torch.float32, device=DEV)
    rng = np.random.default_rng(S)
    pos0 = 0
    for step in range(1 + T):
        q = S if step == 0 else 1
        q32 = rng.standard_normal((B * q, Hq * Dh)).astype(np.float32)
        k32 = rng.standard_normal((B * q, Hkv * Dh)).astype(np.float32)
        v32 = rng.standard_normal((B * q, Hkv * Dh)).astype(np.float32)
        qb = torch.empty(B * q, Hq * Dh, dtype=torch.bfloat16, device=DEV)
        ob = torch.empty(B * q, Hq * Dh, dtype=torch.bfloat16, device=DEV)
        tb.k_rope_kv(torch.from_numpy(q32).to(DEV), torch.from_numpy(k32).to(DEV), torch.from_numpy(v32).to(DEV), qb, kt, vt, cos, sin, mc, B, q, pos0)
        tb.k_attn(qb, kt, vt, ob, mc, B, q, pos0, scratch)
        torch.cuda.synchronize()
        # oracle: same steps
        qo = bf16_round(o.rope(q32.reshape(B, q, Hq, Dh), pos0))
        ko = bf16_round(o.rope(k32.reshape(B, q, Hkv, Dh), pos0))
        vo = bf16_round(v32.reshape(B, q, Hkv, Dh))
        o.K[0, :, :, pos0:pos0 + q] = ko.transpose(0, 2, 1, 3)
        o.V[0, :, :, pos0:pos0 + q] = vo.transpose(0, 2, 1, 3)
        bf16_close(qb.float().cpu().numpy().reshape(B, q, Hq, Dh), qo)
        got_k = tiles_to_cache(kt, cfg, B)[:, :, :pos0 + q]
        bf16_close(got_k, o.K[0, :, :, :pos0 + q])
        assert np.array_equal(tiles_to_cache(vt, cfg, B)[:, :, :pos0 + q], o.V[0, :, :, :pos0 + q].astype(np.float32))
        # attention on the oracle's own q and cache would differ by the rare rounding flips above; feed it the GPU's
        o.K[0, :, :, :pos0 + q] = got_k
        att = o.attention(0, qb.float().cpu().numpy().reshape(B, q, Hq, Dh), pos0)
        got = ob.float().cpu().numpy().reshape(B, q, Hq, Dh)
        assert np.abs(got - att).max() < 2.0 ** -7 * np.abs(att).max() + 1e-6
        assert np.mean(np.abs(got - bf16_round(att))) < 3e-3 * np.abs(att).mean()     # incl. the kernel's bf16 rounding of softmax weights
        pos0 += q
    tb.k_attn_select(0)


@pytest.mark.parametrize("Dh,Hq,Hkv,TK,S,B", [(64, 32, 8, 128, 512, 1), (128, 8, 2, 256, 300, 2), (64, 4, 4, 16, 100, 3)])
def test_tensor_core_prefill_attention_agrees_with_cuda_core_kernel(Dh, Hq, Hkv, TK, S, B):
    """Same q and KV tiles through all three prefill kernels.  The tensor-core kernels round the softmax weights to bf16
    before the second product (its one rounding the oracle does not mirror); outputs are bf16, so agreement is to a
    bf16 ulp, with a small mean difference."""
    cfg = replace(KCFG, Dh=Dh, Hq=Hq, Hkv=Hkv, TK=TK, S=S, T=0, B=B, d=Hq * Dh)
    mc = model_cfg(cfg)
    kt, vt = make_tiles(cfg, B)
    for j, (k, v) in enumerate(zip(kt, vt)):
        k.copy_(bf16_dev(rnd_bits(300 + j, k.numel())) * 30)
        v.copy_(bf16_dev(rnd_bits(400 + j, v.numel())) * 30)
    qb = (bf16_dev(rnd_bits(9, B * S * Hq * Dh)) * 30).view(B * S, Hq * Dh)
    outs = []
    for impl in (3, 2, 1):
        tb.k_attn_select(impl)
        ob = torch.zeros(B * S, Hq * Dh, dtype=torch.bfloat16, device=DEV)
        tb.k_attn(qb, kt, vt, ob, mc, B, S, 0, None)
        torch.cuda.synchronize()
        outs.append(ob.float().cpu().numpy())
    tb.k_attn_select(0)
    assert tb.k_attn_status() == 0
    ref = outs[2]
    assert np.abs(ref).max() > 0
    for a in outs[:2]:                                     # tcgen05 kernel, mma.sync kernel against the CUDA-core kernel
        assert np.isfinite(a).all()
        assert np.abs(a - ref).max() <= 2.0 ** -6 * np.abs(ref).max()
        assert np.abs(a - ref).mean() < 4e-3 * np.abs(ref).mean()


@pytest.mark.parametrize("Dh", [64, 128])
def test_tensor_core_prefill_attention_with_growing_scores(Dh):
    """Scores that grow along the sequence by far more than 2^8 per key block: the tcgen05 kernel has to move its
    exponent reference and rescale its TMEM accumulator at almost every block.  Checked against the oracle."""
    B, Hq, Hkv, TK, S = 2, 4, 2, 64, 400
    cfg = replace(KCFG, Dh=Dh, Hq=Hq, Hkv=Hkv, TK=TK, S=S, T=0, B=B, d=Hq * Dh)
    mc = model_cfg(cfg)
    o = OracleModel(cfg, {(k, 0, -1): rnd_bits(k, 8).reshape(1, 8) for k in range(13)})
    rng = np.random.default_rng(Dh)
    u = rng.standard_normal(Dh).astype(np.float32)
    u /= np.linalg.norm(u)
    ramp = (np.arange(S, dtype=np.float32) / 4.0)[None, None, :, None]                  # + ~16 in log2 units per 64 keys
    k32 = bf16_round(rng.standard_normal((B, Hkv, S, Dh)).astype(np.float32) + ramp * u)
    v32 = bf16_round(rng.standard_normal((B, Hkv, S, Dh)).astype(np.float32))
    q32 = bf16_round(rng.standard_normal((B, S, Hq, Dh)).astype(np.float32) + np.sqrt(Dh).astype(np.float32) * u)
    sgn = np.where(np.arange(Hq) % 2 == 0, 1.0, -1.0).astype(np.float32)[None, None, :, None]
    q32 = q32 * sgn                                                                     # odd heads: scores fall instead
    kt, vt = make_tiles(cfg, B)
    for t in range(cfg.n_tiles):
        lo, hi = t * TK, min(S, (t + 1) * TK)
        kt[t].view(B, Hkv, TK, Dh)[:, :, :hi - lo].copy_(torch.from_numpy(k32[:, :, lo:hi]).to(DEV))
        vt[t].view(B, Hkv, TK, Dh)[:, :, :hi - lo].copy_(torch.from_numpy(v32[:, :, lo:hi]).to(DEV))
    o.K[0, :, :, :S] = k32
    o.V[0, :, :, :S] = v32
    att = o.attention(0, q32, 0)
    qb = torch.from_numpy(q32.reshape(B * S, Hq * Dh)).to(DEV).bfloat16()
    for impl in (3, 2):
        tb.k_attn_select(impl)
        ob = torch.zeros(B * S, Hq * Dh, dtype=torch.bfloat16, device=DEV)
        tb.k_attn(qb, kt, vt, ob, mc, B, S, 0, None)
        torch.cuda.synchronize()
        got = ob.float().cpu().numpy().reshape(B, S, Hq, Dh)
        assert np.isfinite(got).all()
        assert np.abs(got - att).max() < 2.0 ** -6 * np.abs(att).max() + 1e-6
        assert np.mean(np.abs(got - bf16_round(att))) < 4e-3 * np.abs(att).mean()
    tb.k_attn_select(0)
    assert tb.k_attn_status() == 0


@pytest.mark.parametrize("Dh,TK", [(128, 64), (64, 128)])
def test_tensor_core_prefill_attention_of_a_later_chunk(Dh, TK):
    """A prompt processed in two chunks: the second chunk's queries start at position 192 and see the first chunk's keys
    unmasked plus their own causally.  Both tensor-core kernels against the oracle."""
    B, Hq, Hkv, P0, Q2 = 2, 4, 2, 192, 200
    S = P0 + Q2
    cfg = replace(KCFG, Dh=Dh, Hq=Hq, Hkv=Hkv, TK=TK, S=S, T=0, B=B, d=Hq * Dh)
    mc = model_cfg(cfg)
    o = OracleModel(cfg, {(k, 0, -1): rnd_bits(k, 8).reshape(1, 8) for k in range(13)})
    rng = np.random.default_rng(7 * Dh + TK)
    k32 = bf16_round(rng.standard_normal((B, Hkv, S, Dh)).astype(np.float32))
    v32 = bf16_round(rng.standard_normal((B, Hkv, S, Dh)).astype(np.float32))
    q32 = bf16_round(rng.standard_normal((B, Q2, Hq, Dh)).astype(np.float32))
    kt, vt = make_tiles(cfg, B)
    for t in range(cfg.n_tiles):
        lo, hi = t * TK, min(S, (t + 1) * TK)
        if lo < hi:
            kt[t].view(B, Hkv, TK, Dh)[:, :, :hi - lo].copy_(torch.from_numpy(k32[:, :, lo:hi]).to(DEV))
            vt[t].view(B, Hkv, TK, Dh)[:, :, :hi - lo].copy_(torch.from_numpy(v32[:, :, lo:hi]).to(DEV))
    o.K[0, :, :, :S] = k32
    o.V[0, :, :, :S] = v32
    att = o.attention(0, q32, P0)
    qb = torch.from_numpy(q32.reshape(B * Q2, Hq * Dh)).to(DEV).bfloat16()
    for impl in (3, 2):
        tb.k_attn_select(impl)
        ob = torch.zeros(B * Q2, Hq * Dh, dtype=torch.bfloat16, device=DEV)
        tb.k_attn(qb, kt, vt, ob, mc, B, Q2, P0, None)
        torch.cuda.synchronize()
        got = ob.float().cpu().numpy().reshape(B, Q2, Hq, Dh)
        assert np.abs(got - att).max() < 2.0 ** -7 * np.abs(att).max() + 1e-6
        assert np.mean(np.abs(got - bf16_round(att))) < 3e-3 * np.abs(att).mean()
    tb.k_attn_select(0)
    assert tb.k_attn_status() == 0


@pytest.mark.parametrize("Dh,Hq,Hkv,TK,kvlen,B", [(128, 32, 8, 256, 1280, 2), (128, 32, 8, 256, 1037, 3), (128, 64, 8, 64, 2112, 2), (64, 32, 8, 128, 640, 1),
                                                 (64, 4, 4, 16, 48, 1), (128, 8, 4, 32, 33, 2), (64, 8, 1, 16, 17, 4), (128, 4, 4, 48, 1, 2),
                                                 (64, 16, 2, 80, 401, 5)])
def test_tensor_core_decode_attention_matches_oracle_and_cuda_core_kernel(Dh, Hq, Hkv, TK, kvlen, B):
    """Decode attention on the tensor cores (forced wherever the geometry allows) against the oracle's softmax(q K^T) V on
    the same bf16 queries and cache, and against the CUDA-core kernel: contexts that end in the middle of a 16-key chunk,
    span many KV tiles and several CTAs per (sequence, KV head), groups of 1, 2, 4 and 8 query heads, a single key, and
    tiles whose bytes past the context are NaN (they must be neither read into the result nor multiplied by zero)."""
    cfg = replace(KCFG, Dh=Dh, Hq=Hq, Hkv=Hkv, TK=TK, S=kvlen, T=0, B=B, d=Hq * Dh)
    mc = model_cfg(cfg)
    kt, vt = make_tiles(cfg, B)
    assert len(kt) == (kvlen + TK - 1) // TK
    for j, (k, v) in enumerate(zip(kt, vt)):
        k.copy_(bf16_dev(rnd_bits(90 + j, k.numel())) * 40)
        v.copy_(bf16_dev(rnd_bits(190 + j, v.numel())) * 40)
    # everything past the context is poison
    last = kt[-1].view(B, Hkv, TK, Dh), vt[-1].view(B, Hkv, TK, Dh)
    used = kvlen - (len(kt) - 1) * TK
    if used < TK:
        last[0][:, :, used:, :] = float("nan")
        last[1][:, :, used:, :] = float("nan")
    qb = (bf16_dev(rnd_bits(7, B * Hq * Dh)) * 40).view(B, Hq * Dh)
    scratch = torch.empty(tb.k_attn_scratch_bytes(mc) // 4, dtype=torch.float32, device=DEV)
    outs = {}
    for impl in (2, 1):
        tb.k_attn_decode_select(impl)
        ob = torch.full((B, Hq * Dh), float("nan"), dtype=torch.bfloat16, device=DEV)
        tb.k_attn(qb, kt, vt, ob, mc, B, 1, kvlen - 1, scratch)
        torch.cuda.synchronize()
        outs[impl] = ob.float().cpu().numpy().reshape(B, 1, Hq, Dh)
    tb.k_attn_decode_select(0)
    o = OracleModel(cfg, {})
    kc, vc = tiles_to_cache(kt, cfg, B)[:, :, :kvlen], tiles_to_cache(vt, cfg, B)[:, :, :kvlen]
    o.K[0], o.V[0] = kc, vc
    att = o.attention(0, qb.float().cpu().numpy().reshape(B, 1, Hq, Dh), kvlen - 1)
    for impl, got in outs.items():
        assert np.isfinite(got).all(), impl
        assert np.abs(got - att).max() < 2.0 ** -7 * np.abs(att).max() + 1e-6, impl
        assert np.mean(np.abs(got - bf16_round(att))) < 3e-3 * np.abs(att).mean(), impl


def test_attention_single_key_returns_v():
    cfg = replace(KCFG, B=1, S=1, T=0)
    mc = model_cfg(cfg)
    kt, vt = make_tiles(cfg, 1)
    vt[0].copy_(bf16_dev(rnd_bits(9, vt[0].numel())))
    kt[0].copy_(bf16_dev(rnd_bits(8, kt[0].numel())))
    qb = bf16_dev(rnd_bits(7, cfg.Hq * cfg.Dh)).view(1, -1)
    for scratch in (None, torch.empty(tb.k_attn_scratch_bytes(mc) // 4, dtype=torch.float32, device=DEV)):
        ob = torch.empty(1, cfg.Hq * cfg.Dh, dtype=torch.bfloat16, device=DEV)
        tb.k_attn(qb, kt, vt, ob, mc, 1, 1, 0, scratch)
        torch.cuda.synchronize()
        v = vt[0].view(1, cfg.Hkv, cfg.TK, cfg.Dh)[0, :, 0]                     # first token of each kv head
        want = v.repeat_interleave(cfg.Hq // cfg.Hkv, dim=0).reshape(1, -1)
        assert torch.equal(ob, want)


def test_swiglu_and_argmax():
    n = 4 * 1000 + 4
    rng = np.random.default_rng(4)
    g = (rng.standard_normal(n) * 4).astype(np.float32)
    u = rng.standard_normal(n).astype(np.float32)
    out = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    tb.k_swiglu(torch.from_numpy(g).to(DEV), torch.from_numpy(u).to(DEV), out, n)
    torch.cuda.synchronize()
    gd = g.astype(np.float64)
    bf16_close(out.float().cpu().numpy(), bf16_round((gd / (1 + np.exp(-gd)) * u).astype(np.float32)))
    B, V = 5, 128256
    lg = rng.standard_normal((B, V)).astype(np.float32)
    lg[1, 77] = lg[1, 90000] = 9.0            # tie: lowest index wins
    lg[2, :] = 0.5                            # all equal -> 0
    lg[3, V - 1] = 11.0                       # last element
    am = torch.empty(B, dtype=torch.int32, device=DEV)
    tb.k_argmax(torch.from_numpy(lg).to(DEV), am, B, V)
    torch.cuda.synchronize()
    assert am.cpu().numpy().tolist() == np.argmax(lg, axis=1).tolist()
    assert am.cpu().numpy()[1] == 77 and am.cpu().numpy()[2] == 0 and am.cpu().numpy()[3] == V - 1


def test_overlapping_gemv_launches_keep_their_dependencies():
    """Back-to-back weight-streaming launches accumulate into the same output (each depends on the one before through C).
    With dependent-launch overlap a launch starts loading weights early but must not touch C before its predecessor has
    finished: the chain must give bit-identical results with overlap on and off, and equal the oracle's sum."""
    M, n, K, reps = 2, 4100, 2048, 12
    a_bits = rnd_bits(21, M * K).reshape(M, K)
    A = bf16_dev(a_bits)
    Ws = [rnd_bits(30 + i, n * K).reshape(n, K) for i in range(3)]
    Wd = [bf16_dev(w) for w in Ws]
    outs = []
    for overlap in (1, 0):
        tb.k_gemv_overlap(overlap)
        Cd = torch.zeros(M, n, dtype=torch.float32, device=DEV)
        for i in range(reps):
            tb.k_gemm(A, Wd[i % 3], Cd, M, n, K, n, 0, 1)
        torch.cuda.synchronize()
        outs.append(Cd.cpu().numpy())
    tb.k_gemv_overlap(1)
    assert np.array_equal(outs[0], outs[1])
    o = oracle()
    a = si.bf16_bits_to_f32(a_bits)
    want = sum(o.linear(a, si.bf16_bits_to_f32(Ws[i % 3]).astype(np.float64)).astype(np.float64) for i in range(reps))
    assert np.abs(outs[0] - want).max() < 1e-4 * np.abs(want).max()


def test_chained_products_read_their_activations_early_with_the_same_bits():
    """Under the caller's promise (tgp_k_gemm_chain) a product that directly follows another one over the same activations
    requests them before its predecessor has finished.  The chain must give the bits of unchained launches; a product
    that follows a kernel which rewrote the activations (an RMSNorm of this library) is not chained and sees the new values."""
    M, n, K = 8, 1152, 4096
    rng = np.random.default_rng(77)
    x0 = torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).to(DEV)
    gain = bf16_dev(rnd_bits(78, K))
    A = torch.empty(M, K, dtype=torch.bfloat16, device=DEV)
    Ws = [bf16_dev(rnd_bits(80 + i, n * K).reshape(n, K)) for i in range(4)]
    outs = []
    for chain in (0, 1):
        tb.k_gemm_chain(chain)
        x = x0.clone()
        res = []
        for rep in range(3):
            tb.k_rmsnorm(x, K, gain, A, M, K, 1e-5)               # rewrites A: the product after it waits for it
            x.mul_(1.25)                                          # (another stream op between the repetitions; before the norm, not between products)
            Cs = [torch.zeros(M, n, dtype=torch.float32, device=DEV) for _ in Ws]
            for W, C in zip(Ws, Cs):
                tb.k_gemm(A, W, C, M, n, K, n, 0, 0)
            torch.cuda.synchronize()
            res.append([c.cpu().numpy() for c in Cs])
        outs.append(res)
    tb.k_gemm_chain(0)
    for rep in range(3):
        for a, b in zip(outs[0][rep], outs[1][rep]):
            assert np.array_equal(a, b)
    assert not np.array_equal(outs[0][0][0], outs[0][1][0])          # the activations did change between repetitions


@pytest.mark.parametrize("M,ns,K,grouped", [
    (1, (2048, 512, 512), 2048, True),            # the q, k, v projections of the 1B shape: one launch
    (2, (300, 7, 129, 1), 264, True),             # four ragged parts, K not a multiple of the chunk
    (1, (4096, 8192), 4096, False),               # a block of many rows is launched alone
    (2, (640, 640, 64), 8192, False),             # long K at M <= 2: the parts take the split-K kernel, alone
    (8, (1152, 1152, 1152, 640), 14336, True),    # the pieces of an 8B down projection: 8-row CTAs, 16 warps
    (16, (512,) * 8, 28672, True),                # eight pieces of a 70B down projection
    (8, (1024, 1024), 4096, True),                # k and v of the 8B shape
    (8, (4096, 1024, 1024), 4096, True),          # q, k and v of the 8B shape: all take the persistent 16-warp kernel
    (8, (4096, 4096, 4096, 2048, 4096, 4096, 4096, 2048), 4096, True),   # gate and up of the 8B shape in 32 MiB pieces
    (8, (8192, 1024), 2048, False),               # a piece of many rows takes the 8-warp kernel: one launch each
    (32, (500, 260, 33), 160, True),              # ragged row counts, four groups of activation rows
    (5, (24000, 64), 64, False),                  # a block that fills the machine alone
    (40, (256, 256), 512, False)])                # more activation rows than the skinny kernels take
@pytest.mark.parametrize("accumulate", [0, 1])
def test_grouped_products_equal_single_products_and_oracle(M, ns, K, grouped, accumulate):
    """Products that share their activations: the grouped call must give the bits of one tgp_k_gemm() call per part,
    whether it runs as one launch or falls back to one launch per part, with the switch on and off, and leave the
    columns beyond each part untouched; the values are checked against the oracle's linear()."""
    keys = {tb.k_gemm_group_key(M, n, K) for n in ns}
    assert (len(keys) == 1 and 0 not in keys) == grouped
    a_bits = rnd_bits(51, M * K).reshape(M, K)
    A = bf16_dev(a_bits)
    w_bits = [rnd_bits(60 + s, n * K).reshape(n, K) for s, n in enumerate(ns)]
    Wd = [bf16_dev(w) for w in w_bits]
    ldcs = [n + 8 * (s + 1) for s, n in enumerate(ns)]
    c0 = [np.random.default_rng(100 + s).standard_normal((M, ld)).astype(np.float32) * 0.01 for s, ld in enumerate(ldcs)]
    fresh = lambda: [torch.from_numpy(c.copy()).to(DEV) for c in c0]
    single = fresh()
    for s, n in enumerate(ns):
        tb.k_gemm(A, Wd[s], single[s], M, n, K, ldcs[s], 0, accumulate)
    outs = []
    for enable in (1, 0):
        tb.k_gemm_group_select(enable)
        out = fresh()
        tb.k_gemm_group(A, Wd, out, M, list(ns), K, ldcs, accumulate)
        torch.cuda.synchronize()
        outs.append([g.cpu().numpy() for g in out])
        assert enable or tb.k_gemm_group_key(M, ns[0], K) == 0
    tb.k_gemm_group_select(1)
    o = oracle()
    a = si.bf16_bits_to_f32(a_bits)
    for s, n in enumerate(ns):
        ref = single[s].cpu().numpy()
        assert np.array_equal(outs[0][s], ref) and np.array_equal(outs[1][s], ref)
        assert np.array_equal(ref[:, n:], c0[s][:, n:])
        want = o.linear(a, si.bf16_bits_to_f32(w_bits[s]).astype(np.float64)).astype(np.float64) + (c0[s][:, :n] if accumulate else 0)
        assert np.abs(ref[:, :n] - want).max() < 2e-5 * max(np.abs(want).max(), 0.01) + 1e-7
    if M == 1 and accumulate == 0:
        with pytest.raises(tb.TgpError):
            tb.k_gemm_group(A, Wd[:1] * 9, [single[0]] * 9, M, [ns[0]] * 9, K, [ldcs[0]] * 9)      # more parts than the call takes
        with pytest.raises(tb.TgpError):
            tb.k_gemm_group(A, Wd[:2], single[:2], M, [ns[0], ns[1]], K, [ns[0] - 1, ldcs[1]])       # row stride below the part's width


@pytest.mark.parametrize("M,n,K", [(3, 100, 64), (8, 4096, 4096), (8, 1030, 512), (13, 77, 128), (16, 260, 1024), (17, 64, 96), (24, 2049, 2048),
                                   (32, 4100, 8192), (5, 16, 32),
                                   # few rows and long K: the split-K kernel (K divided among the warps of a CTA; ragged rows, K that
                                   # leaves the last warps without a chunk)
                                   (8, 1152, 14336), (5, 650, 14368), (16, 1024, 4096), (9, 24, 2080), (8, 16, 16384)])
@pytest.mark.parametrize("accumulate", [0, 1])
def test_skinny_tensor_core_gemv_matches_oracle_and_cuda_core_path(M, n, K, accumulate):
    a_bits, w_bits = rnd_bits(41, M * K).reshape(M, K), rnd_bits(42, n * K).reshape(n, K)
    A, W = bf16_dev(a_bits), bf16_dev(w_bits)
    c0 = np.random.default_rng(M + n).standard_normal((M, n + 8)).astype(np.float32) * 0.01
    outs = []
    for impl in (0, 1):
        tb.k_skinny_select(impl)
        Cd = torch.from_numpy(c0.copy()).to(DEV)
        tb.k_gemm(A, W, Cd, M, n, K, n + 8, 4, accumulate)
        torch.cuda.synchronize()
        outs.append(Cd.cpu().numpy())
    tb.k_skinny_select(0)
    want = c0.astype(np.float64).copy()
    prod = oracle().linear(si.bf16_bits_to_f32(a_bits), si.bf16_bits_to_f32(w_bits).astype(np.float64)).astype(np.float64)
    want[:, 4:4 + n] = prod + (c0[:, 4:4 + n] if accumulate else 0)
    scale = max(np.abs(prod).max(), 0.01)
    assert np.abs(outs[0] - want).max() < 2e-5 * scale + 1e-7
    assert np.abs(outs[0] - outs[1]).max() < 2e-5 * scale + 1e-7
    for out in outs:
        assert np.array_equal(out[:, :4], c0[:, :4]) and np.array_equal(out[:, 4 + n:], c0[:, 4 + n:])
