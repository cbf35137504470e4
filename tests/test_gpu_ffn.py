"""GPU parity of hidden RMSNorm, fused residual + RMSNorm, SwiGLU and the dense linear layer
against the CPU oracle, and their bit-identity between batched and row-by-row use (the paper's
operator table verifies each of them bitwise between full-sequence and token-wise execution)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_common import count_diff

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _randn(shape, seed, std=1.0):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return (torch.randn(shape, generator=g, device="cuda") * std).to(torch.bfloat16)


def _close_bf16(got, ref, abs_tol=1e-6):
    g = got.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(g - ref) <= 2.0 ** -8 * np.abs(ref) + abs_tol), float(np.abs(g - ref).max())


@pytest.mark.parametrize("H", [8, 64, 1000, 1536, 3584, 4096, 5120, 8192])
def test_rmsnorm_matches_oracle_and_rows_are_independent(tik, H):
    T = 37
    x = _randn((T, H), 500 + H, 2.0)
    w = (1 + 0.2 * _randn((H,), 600 + H).float()).to(torch.bfloat16)
    y = tik.tik_rmsnorm(x, w, 1e-6)
    _close_bf16(y, oracle.rmsnorm(x.float().cpu().numpy(), w.float().cpu().numpy(), 1e-6))
    for a, b in [(0, 1), (5, 6), (30, 37)]:
        assert count_diff(tik.tik_rmsnorm(x[a:b].contiguous(), w, 1e-6), y[a:b]) == 0
    # in place
    x2 = x.clone()
    tik.tik_rmsnorm(x2, w, 1e-6, y=x2)
    assert count_diff(x2, y) == 0


@pytest.mark.parametrize("H", [64, 1536, 4096, 8192])
def test_fused_residual_rmsnorm(tik, H):
    T = 29
    x = _randn((T, H), 700 + H)
    res0 = _randn((T, H), 800 + H, 20.0)
    w = (1 + 0.2 * _randn((H,), 900 + H).float()).to(torch.bfloat16)
    res = res0.clone()
    y = tik.tik_rmsnorm(x, w, 1e-6, residual=res)
    y_ref, s_ref = oracle.rmsnorm(x.float().cpu().numpy(), w.float().cpu().numpy(), 1e-6,
                                  residual=res0.float().cpu().numpy())
    assert np.array_equal(res.float().cpu().numpy(), s_ref)         # the stored sum, bit for bit
    assert count_diff(res, x + res0) == 0                           # == a bf16 tensor add
    _close_bf16(y, y_ref)
    assert count_diff(y, tik.tik_rmsnorm(res, w, 1e-6)) == 0        # fused == add, then plain norm
    # token-wise == batched
    r1 = res0[3:4].clone()
    y1 = tik.tik_rmsnorm(x[3:4].contiguous(), w, 1e-6, residual=r1)
    assert count_diff(y1, y[3:4]) == 0 and count_diff(r1, res[3:4]) == 0


@pytest.mark.parametrize("T,I", [(1, 8), (33, 1000), (257, 8960), (64, 18944), (1100, 8960)])   # the last one: four vectors per thread, ragged last block
def test_swiglu(tik, T, I):
    gu = _randn((T, 2 * I), 1000 + I, 3.0)
    gu[0, :4] = torch.tensor([0.0, 40.0, -40.0, -100.0], dtype=torch.bfloat16)
    out = tik.tik_swiglu(gu)
    _close_bf16(out, oracle.swiglu(gu.float().cpu().numpy()), abs_tol=1e-5)
    assert bool(torch.isfinite(out).all())
    t = T // 2
    assert count_diff(tik.tik_swiglu(gu[t:t + 1].contiguous()), out[t:t + 1]) == 0


@pytest.mark.parametrize("T,K,N", [(1, 64, 8), (300, 1536, 1000), (129, 8960, 1536), (700, 1536, 2304),
                                   (4100, 256, 1032)])
def test_linear_matches_oracle_and_is_batch_invariant(tik, T, K, N):
    x = _randn((T, K), 1100 + K)
    W = _randn((N, K), 1200 + N, 0.02)
    y = tik.tik_linear(x, W)
    ref = oracle.linear(x.float().cpu().numpy(), W.float().cpu().numpy())
    g = y.float().cpu().numpy().astype(np.float64)
    scale = 0.02 * np.sqrt(K)
    assert np.all(np.abs(g - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4 * scale), float(np.abs(g - ref).max())
    # a row alone (decode), a ragged slice and a slice that starts inside a 128-row tile
    for a, b in [(0, 1), (T - 1, T), (T // 3, T // 3 + 5), (max(0, T - 131), T)]:
        if a < b:
            assert count_diff(tik.tik_linear(x[a:b].contiguous(), W), y[a:b]) == 0, (a, b)
    # canary: nothing is written outside [T][N]
    buf = torch.full((T + 2, N), -7.0, dtype=torch.bfloat16, device="cuda")
    tik.tik_linear(x, W, y=buf[1:T + 1])
    assert bool((buf[0] == -7.0).all()) and bool((buf[T + 1] == -7.0).all())
    assert count_diff(buf[1:T + 1], y) == 0


@pytest.mark.parametrize("K,N", [(512, 37888), (256, 55296), (1024, 5120), (192, 1000), (128, 72), (64, 40000),
                                 (27648, 5120), (3584, 37888)])
def test_decode_shaped_linear_equals_rows_of_a_batched_call(tik, K, N):
    """One row tile (T <= 128) takes the persistent column-unit schedule with 64, 128 or 256 columns
    per unit and 32, 64 or 128 staged rows; every such call returns the bits of the same rows inside a
    300-row call (CTA pairs, 256-column steps), and writes nothing outside its [T][N] block.  Two row
    tiles (T <= 256) run the pair kernel persistently over 256-column steps: same check."""
    x = _randn((300, K), 2100 + K)
    W = _randn((N, K), 2200 + N % 977, 0.02)
    y = tik.tik_linear(x, W)
    ncol = min(N, 4096)                   # the oracle on three rows and the first columns (full-size K x N: seconds)
    ref = oracle.linear(x[:3].float().cpu().numpy(), W[:ncol].float().cpu().numpy())
    g = y[:3, :ncol].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(g - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4 * 0.02 * np.sqrt(K))
    for a, T in [(0, 1), (7, 16), (100, 32), (3, 33), (50, 64), (171, 65), (172, 128), (90, 129), (20, 200), (44, 256)]:
        buf = torch.full((T + 2, N), -7.0, dtype=torch.bfloat16, device="cuda")
        tik.tik_linear(x[a:a + T].contiguous(), W, y=buf[1:T + 1])
        assert count_diff(buf[1:T + 1], y[a:a + T]) == 0, (a, T)
        assert bool((buf[0] == -7.0).all()) and bool((buf[T + 1] == -7.0).all())
    assert tik.device_status() == 0


def test_ffn_block_composition(tik):
    """norm -> gate/up projection -> SwiGLU -> down projection, batched and token by token."""
    T, H, I = 70, 512, 1408
    x = _randn((T, H), 1)
    res = _randn((T, H), 2)
    w = (1 + 0.1 * _randn((H,), 3).float()).to(torch.bfloat16)
    Wgu, Wd = _randn((2 * I, H), 4, 0.03), _randn((H, I), 5, 0.03)

    def block(xs, rs):
        r = rs.clone()
        h = tik.tik_rmsnorm(xs, w, 1e-6, residual=r)
        return tik.tik_linear(tik.tik_swiglu(tik.tik_linear(h, Wgu)), Wd), r

    y, r = block(x, res)
    for t in (0, 17, 69):
        y1, r1 = block(x[t:t + 1].contiguous(), res[t:t + 1].contiguous())
        assert count_diff(y1, y[t:t + 1]) == 0 and count_diff(r1, r[t:t + 1]) == 0
    # against the oracle chain evaluated on the GPU's own intermediate roundings
    h_ref, s = oracle.rmsnorm(x.float().cpu().numpy(), w.float().cpu().numpy(), 1e-6, residual=res.float().cpu().numpy())
    h = tik.tik_rmsnorm(x, w, 1e-6, residual=res.clone())
    _close_bf16(h, h_ref)
    gu = tik.tik_linear(h, Wgu)
    a = tik.tik_swiglu(gu)
    _close_bf16(a, oracle.swiglu(gu.float().cpu().numpy()), abs_tol=1e-5)
    ref = oracle.linear(a.float().cpu().numpy(), Wd.float().cpu().numpy())
    g = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(g - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-3)


def test_ffn_invalid_arguments(tik):
    x = _randn((4, 64), 1)
    w = _randn((64,), 2)
    with pytest.raises(tik.TikError):
        tik.tik_rmsnorm(_randn((4, 12), 1), _randn((12,), 2), 1e-6)          # H % 8
    with pytest.raises(tik.TikError):
        tik.tik_rmsnorm(x, w, -1.0)
    with pytest.raises(tik.TikError):
        tik.tik_linear(_randn((4, 32), 1), _randn((8, 32), 2))                # K % 64
    with pytest.raises(tik.TikError):
        tik.tik_linear(x, _randn((12, 64), 2))                                # N % 8
    with pytest.raises(tik.TikError):
        tik.tik_swiglu(_randn((4, 24), 1))                                    # I % 8
    assert tik.tik_linear(x[:0], _randn((8, 64), 2)).shape == (0, 8)
