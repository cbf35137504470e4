"""GPU parity: token log-probabilities against the CPU oracle and across batch shapes."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth
from gpu_common import LOGPROB_TOL, bits, count_diff

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _inputs(T, H, V, seed, std=0.02):
    g = torch.Generator(device="cuda").manual_seed(seed)
    hidden = torch.randn(T, H, generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g, device="cuda") * std).to(torch.bfloat16)
    target = torch.randint(0, V, (T,), generator=g, device="cuda").to(torch.int32)
    return hidden, W, target


def _oracle(hidden, W, target, inv_t=1.0):
    return oracle.token_logprob(hidden.float().cpu().numpy(), W.float().cpu().numpy(),
                                target.cpu().numpy(), inv_t)


def test_tiny_workload_every_token(tik):
    w = synth.get_workload(0)
    hidden, W, target = synth.make_logprob_inputs(w, "cuda")
    lse = torch.empty(hidden.shape[0], dtype=torch.float32, device="cuda")
    lp = tik.tik_token_logprob(hidden, W, target, lse=lse)
    ref, ref_lse = _oracle(hidden, W, target)
    assert np.abs(lp.cpu().numpy() - ref).max() <= LOGPROB_TOL
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= LOGPROB_TOL


@pytest.mark.parametrize("T,H,V,std,inv_t", [
    (1, 64, 5, 1.0, 1.0),             # a single row, vocabulary smaller than one tile
    (130, 128, 1000, 0.3, 1.0),       # ragged rows and columns inside one super-chunk
    (257, 320, 2500, 0.1, 0.7),       # three token tiles, three super-chunks, temperature
    (64, 1536, 4097, 0.02, 1.0),      # one column into a fifth super-chunk
])
def test_ragged_shapes(tik, T, H, V, std, inv_t):
    hidden, W, target = _inputs(T, H, V, 1234 + T, std)
    target[0] = V - 1
    target[-1] = 0
    lp = tik.tik_token_logprob(hidden, W, target, inv_temperature=inv_t)
    ref, _ = _oracle(hidden, W, target, inv_t)
    assert np.abs(lp.cpu().numpy() - ref).max() <= LOGPROB_TOL


def test_zero_weights_give_minus_ln_v(tik):
    T, H, V = 40, 128, 2048
    hidden, _, target = _inputs(T, H, V, 5)
    W = torch.zeros(V, H, dtype=torch.bfloat16, device="cuda")
    lp = tik.tik_token_logprob(hidden, W, target)
    assert np.abs(lp.cpu().numpy() + math.log(V)).max() <= 1e-5


def test_batch_shape_invariance(tik):
    """The same hidden rows scored in one call, row by row, in permuted order and in
    decode-sized batches give identical bits."""
    T, H, V = 300, 256, 3000
    hidden, W, target = _inputs(T, H, V, 77, 0.2)
    full = tik.tik_token_logprob(hidden, W, target)
    perm = torch.randperm(T, device="cuda", generator=torch.Generator(device="cuda").manual_seed(3))
    permuted = tik.tik_token_logprob(hidden[perm].contiguous(), W, target[perm].contiguous())
    assert count_diff(full[perm], permuted) == 0
    for a, b in [(0, 1), (5, 6), (127, 129), (0, 16), (200, 300), (64, 192)]:
        part = tik.tik_token_logprob(hidden[a:b].contiguous(), W, target[a:b].contiguous())
        assert count_diff(full[a:b], part) == 0, (a, b)


def test_mid_sized_calls_equal_rows_of_a_large_call(tik):
    """Calls of 3 to 16 token tiles run persistently over (vocabulary step, pair of token tiles)
    units with one partial per 128-column tile; a larger call keeps one partial per 1024 columns.
    Same rows, same bits; sampled rows against the oracle."""
    T, H, V = 2500, 192, 5000 + 8
    hidden, W, target = _inputs(T, H, V, 99, 0.3)
    target[:3] = torch.tensor([0, V - 1, 4095], dtype=torch.int32)
    full = tik.tik_token_logprob(hidden, W, target)
    rows = torch.tensor([0, 1, 2, 255, 256, 257, 1023, 1024, 2047, 2048, T - 1], device="cuda")
    ref, _ = _oracle(hidden[rows], W, target[rows])
    assert np.abs(full[rows].cpu().numpy() - ref).max() <= LOGPROB_TOL
    for a, b in [(0, 700), (300, 2348), (1000, 1513), (2100, 2500), (0, 257), (1, 2049)]:
        part = tik.tik_token_logprob(hidden[a:b].contiguous(), W, target[a:b].contiguous())
        assert count_diff(full[a:b], part) == 0, (a, b)


def test_two_bands_several_super_chunks_per_cta(tik):
    """More than one band of 32 token tiles (the second one a single, partner-less tile) and enough
    work that a CTA walks two super-chunks: sampled rows against the oracle, slices bit for bit."""
    T, H, V = 128 * 40 + 70, 64, 32768 + 11
    hidden, W, target = _inputs(T, H, V, 4321, 0.5)
    target[:4] = torch.tensor([0, V - 1, 32767, 32768], dtype=torch.int32)
    lp = tik.tik_token_logprob(hidden, W, target)
    rows = torch.tensor([0, 1, 2, 3, 127, 128, 4095, 4096, 5119, 5120, T - 1] + list(range(900, 5000, 97)), device="cuda")
    ref, _ = _oracle(hidden[rows], W, target[rows])
    assert np.abs(lp[rows].cpu().numpy() - ref).max() <= LOGPROB_TOL
    assert bool(torch.isfinite(lp).all())
    for a, b in [(5120, T), (4000, 4100), (T - 1, T)]:
        part = tik.tik_token_logprob(hidden[a:b].contiguous(), W, target[a:b].contiguous())
        assert count_diff(lp[a:b], part) == 0, (a, b)


def test_bad_target_is_nan_and_flagged(tik):
    T, H, V = 8, 64, 100
    hidden, W, target = _inputs(T, H, V, 9)
    target[3] = V
    target[5] = -1
    lp = tik.tik_token_logprob(hidden, W, target).cpu().numpy()
    assert np.isnan(lp[3]) and np.isnan(lp[5])
    good = [0, 1, 2, 4, 6, 7]
    ref, _ = _oracle(hidden, W, target)
    assert np.abs(lp[good] - ref[good]).max() <= LOGPROB_TOL
    assert tik.device_status() & tik.DEV_BAD_TARGET
