"""Pins for the oracles of the remaining unified operators (hidden RMSNorm, fused residual +
RMSNorm, SwiGLU, dense linear layer): closed forms, identities and library routines in fp64 that a
dropped term, a swapped operand or a transposed index would break."""
import math

import numpy as np
import torch

import oracle


def _bf16(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).float().numpy()


def test_rmsnorm_closed_forms_and_library():
    H = 96
    ones = np.ones(H, dtype=np.float32)
    x = np.full((2, H), -2.0, dtype=np.float32)
    assert np.abs(oracle.rmsnorm(x, ones, 0.5) - (-2.0 / math.sqrt(4.5))).max() < 1e-14
    rng = np.random.default_rng(11)
    x = rng.standard_normal((5, H)).astype(np.float32)
    w = (1 + 0.3 * rng.standard_normal(H)).astype(np.float32)
    y = oracle.rmsnorm(x, w, 1e-6)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (H,), torch.from_numpy(w).double(), 1e-6)
    assert np.abs(y - ref.numpy()).max() < 1e-12
    # rows are independent, eps = 0 is scale invariant, unit weight gives unit mean square
    assert np.array_equal(oracle.rmsnorm(x[2:3], w, 1e-6), y[2:3])
    assert np.abs(oracle.rmsnorm(8 * x, w, 0.0) - oracle.rmsnorm(x, w, 0.0)).max() < 1e-12
    assert np.abs((oracle.rmsnorm(x, ones, 0.0) ** 2).mean(-1) - 1).max() < 1e-12


def test_fused_residual_rmsnorm_is_add_then_norm_of_the_stored_sum():
    rng = np.random.default_rng(12)
    H = 64
    x = _bf16(rng.standard_normal((7, H)))
    r = _bf16(30 * rng.standard_normal((7, H)))            # different magnitudes: the sum really rounds
    w = _bf16(1 + 0.2 * rng.standard_normal(H))
    y, s = oracle.rmsnorm(x, w, 1e-6, residual=r)
    s_ref = (torch.from_numpy(x).to(torch.bfloat16) + torch.from_numpy(r).to(torch.bfloat16)).float().numpy()
    assert np.array_equal(s, s_ref)                       # torch's own bf16 add (fp32 sum, RNE)
    assert np.any(s != x + r)                             # ... and it is not the exact sum
    assert np.array_equal(y, oracle.rmsnorm(s, w, 1e-6))  # fused == unfused
    # zero residual changes nothing
    y0, s0 = oracle.rmsnorm(x, w, 1e-6, residual=np.zeros_like(x))
    assert np.array_equal(s0, x) and np.array_equal(y0, oracle.rmsnorm(x, w, 1e-6))


def test_swiglu_identities_and_library():
    g = np.array([[0.0, 1.0, -1.0, 30.0, -30.0, 0.5]], dtype=np.float32)
    u = np.array([[5.0, 2.0, 2.0, 1.0, 1.0, -4.0]], dtype=np.float32)
    out = oracle.swiglu(np.concatenate([g, u], axis=1))[0]
    assert out[0] == 0.0
    assert abs(out[1] - 2.0 / (1 + math.exp(-1.0))) < 1e-15
    assert abs(out[1] - out[2] - 2.0) < 1e-14             # silu(x) - silu(-x) = x
    assert abs(out[3] - 30.0) < 1e-10 and abs(out[4]) < 1e-10
    assert abs(out[5] - (-4.0) * 0.5 / (1 + math.exp(-0.5))) < 1e-15
    rng = np.random.default_rng(13)
    gu = rng.standard_normal((9, 2 * 40)).astype(np.float32) * 3
    ref = torch.nn.functional.silu(torch.from_numpy(gu[:, :40]).double()) * torch.from_numpy(gu[:, 40:]).double()
    assert np.abs(oracle.swiglu(gu) - ref.numpy()).max() < 1e-13
    # gate and up are not interchangeable, and the split is halves, not interleaved
    swapped = np.concatenate([gu[:, 40:], gu[:, :40]], axis=1)
    assert np.abs(oracle.swiglu(swapped) - oracle.swiglu(gu)).max() > 0.1


def test_linear_against_numpy_identity_and_one_hot():
    rng = np.random.default_rng(14)
    T, K, N = 6, 50, 33
    x = rng.standard_normal((T, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    y = oracle.linear(x, W)
    assert np.abs(y - x.astype(np.float64) @ W.astype(np.float64).T).max() < 1e-12
    assert np.array_equal(oracle.linear(x, np.eye(K, dtype=np.float32)), x.astype(np.float64))
    onehot = np.zeros((1, K), dtype=np.float32)
    onehot[0, 7] = 1.0
    assert np.array_equal(oracle.linear(onehot, W)[0], W[:, 7].astype(np.float64))     # column 7 of W, not row 7
    # homogeneous (scaling by a power of two is exact), rows independent
    assert np.array_equal(oracle.linear(2 * x, W), 2 * y)
    assert np.array_equal(oracle.linear(x[3:4], W), y[3:4])


def test_f32_instantiations_stay_close():
    rng = np.random.default_rng(15)
    x = rng.standard_normal((4, 256)).astype(np.float32)
    w = np.ones(256, dtype=np.float32)
    assert np.abs(oracle.rmsnorm(x, w, 1e-6) - oracle.rmsnorm(x, w, 1e-6, f32=True)).max() < 1e-5
    assert np.abs(oracle.swiglu(x) - oracle.swiglu(x, f32=True)).max() < 1e-5
    W = (0.02 * rng.standard_normal((64, 256))).astype(np.float32)
    assert np.abs(oracle.linear(x, W) - oracle.linear(x, W, f32=True)).max() < 1e-5
