"""Pins for the CPU token log-probability oracle."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed, std=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * std).to(torch.bfloat16).float().numpy()


def _uniform_golden():
    out = []
    with open(os.path.join(GOLDEN, "logprob_uniform.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                V, val = line.split()
                out.append((int(V), float(val)))
    return out


def test_uniform_golden_values_are_minus_ln_v():
    for V, val in _uniform_golden():
        assert abs(val + math.log(V)) < 1e-11


@pytest.mark.parametrize("V,val", _uniform_golden())
def test_zero_weights_give_minus_ln_v(V, val):
    H, T = 8, 3
    hidden = _rand((T, H), 1)
    W = np.zeros((V, H), np.float32)
    target = np.array([0, V // 2, V - 1], np.int32)
    lp, lse = oracle.token_logprob(hidden, W, target)
    assert np.abs(lp - val).max() < 1e-11
    assert np.abs(lse - math.log(V)).max() < 1e-11
    # zero hidden state, random weights: same answer
    lp2, _ = oracle.token_logprob(np.zeros((T, H), np.float32), _rand((V, H), 2), target)
    assert np.abs(lp2 - val).max() < 1e-11


def _closed_form_cases():
    cases = []
    with open(os.path.join(GOLDEN, "logprob_closed_form.txt")) as f:
        for line in f:
            if not line.startswith("case"):
                continue
            parts = [p.split() for p in line[4:].split("|")]
            cases.append((float(parts[0][0]), [int(x) for x in parts[1]], int(parts[2][0]),
                          Fraction(parts[3][0])))
    return cases


@pytest.mark.parametrize("a,w,target,prob", _closed_form_cases())
def test_golden_one_hot_logits(a, w, target, prob):
    V, H = len(w), 5
    hidden = np.zeros((1, H), np.float32)
    hidden[0, 0] = a
    W = np.zeros((V, H), np.float32)
    W[:, 0] = [math.log(x) / a for x in w]
    W[:, 1:] = _rand((V, H - 1), 3)           # multiplied by the zeros of hidden
    lp, lse = oracle.token_logprob(hidden, W, np.array([target], np.int32))
    assert abs(lp[0] - math.log(float(prob))) < 2e-6
    assert abs(lse[0] - math.log(sum(w))) < 2e-6


def test_log_softmax_row_normalises():
    w = synth.get_workload(0)
    hidden, W, target = synth.make_logprob_inputs(w)
    hidden, W, target = hidden.float().numpy(), W.float().numpy(), target.numpy()
    for t in (0, 17, 127):
        row = oracle.log_softmax_row(hidden[t], W)
        assert row.shape == (w.vocab,)
        assert (row <= 0).all()
        assert abs(np.exp(row).sum() - 1.0) < 1e-12
    lp, lse = oracle.token_logprob(hidden, W, target)
    for t in (0, 17, 127):
        row = oracle.log_softmax_row(hidden[t], W)
        assert lp[t] == row[target[t]]


def test_matches_library_log_softmax():
    T, H, V = 9, 48, 301
    hidden, W = _rand((T, H), 4), _rand((V, H), 5, 0.3)
    target = np.arange(T, dtype=np.int32) * 31 % V
    lp, lse = oracle.token_logprob(hidden, W, target, inv_temperature=0.7)
    z = torch.from_numpy(hidden).double() @ torch.from_numpy(W).double().T * 0.7
    ref = torch.log_softmax(z, dim=-1).gather(1, torch.from_numpy(target).long()[:, None])[:, 0]
    np.testing.assert_allclose(lp, ref.numpy(), atol=1e-11)
    np.testing.assert_allclose(lse, torch.logsumexp(z, -1).numpy(), atol=1e-11)


def test_brute_force_tiny():
    T, H, V = 3, 4, 7
    hidden, W = _rand((T, H), 6), _rand((V, H), 7)
    target = np.array([6, 0, 3], np.int32)
    lp, _ = oracle.token_logprob(hidden, W, target)
    for t in range(T):
        z = []
        for v in range(V):
            acc = 0.0
            for c in range(H):
                acc += float(hidden[t, c]) * float(W[v, c])
            z.append(acc)
        den = sum(math.exp(x) for x in z)
        assert abs(lp[t] - math.log(math.exp(z[target[t]]) / den)) < 1e-12


def test_temperature_and_shift_invariance():
    T, H, V = 5, 16, 64
    hidden, W = _rand((T, H), 8), _rand((V, H), 9, 0.5)
    target = np.array([1, 5, 9, 33, 63], np.int32)
    a, _ = oracle.token_logprob(hidden, W, target, inv_temperature=0.5)
    b, _ = oracle.token_logprob(hidden * 0.5, W, target)      # scaling by 2^-1 is exact
    np.testing.assert_allclose(a, b, atol=1e-13)
    # a constant added to every logit (extra coordinate with equal weights) cancels
    h2 = np.concatenate([hidden, np.ones((T, 1), np.float32)], 1)
    W2 = np.concatenate([W, np.full((V, 1), 3.0, np.float32)], 1)
    c, lse_c = oracle.token_logprob(h2, W2, target)
    d, lse_d = oracle.token_logprob(hidden, W, target)
    np.testing.assert_allclose(c, d, atol=1e-12)
    np.testing.assert_allclose(lse_c, lse_d + 3.0, atol=1e-12)


def test_rows_are_independent_and_bad_target_is_nan():
    T, H, V = 6, 8, 32
    hidden, W = _rand((T, H), 10), _rand((V, H), 11)
    target = np.array([0, 31, 32, -1, 4, 5], np.int32)
    lp, _ = oracle.token_logprob(hidden, W, target)
    assert np.isnan(lp[2]) and np.isnan(lp[3]) and np.isfinite(lp[[0, 1, 4, 5]]).all()
    one, _ = oracle.token_logprob(hidden[4:5], W, target[4:5])
    assert one[0] == lp[4]


def test_fp32_arithmetic_variant_is_close():
    w = synth.get_workload(0)
    hidden, W, target = synth.make_logprob_inputs(w)
    a, _ = oracle.token_logprob(hidden.float().numpy(), W.float().numpy(), target.numpy())
    b, _ = oracle.token_logprob(hidden.float().numpy(), W.float().numpy(), target.numpy(),
                                f32=True)
    assert np.abs(a - b).max() < 1e-4
