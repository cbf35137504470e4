"""Pins for the oracle of the pre-attention step (RMSNorm -> NeoX RoPE -> indexed cache write):
each is something the mathematics fixes independently of the oracle's own loops -- rotation as a
complex product, invariants, closed forms, a library routine on a textbook case."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth


def _table(max_pos, d, base=10000.0):
    return synth.make_rope_table(max_pos, d, base).numpy()


def test_rope_table_entries_and_angle_addition():
    tab = _table(64, 4, 10000.0).astype(np.float64)
    # d = 4, base 1e4: theta = (1, 0.01)
    assert tab[0].tolist() == [1.0, 1.0, 0.0, 0.0]
    assert abs(tab[2, 0] - (-0.4161468365471424)) < 1e-7      # cos 2
    assert abs(tab[2, 2] - 0.9092974268256817) < 1e-7         # sin 2
    assert abs(tab[50, 1] - 0.8775825618903728) < 1e-7        # cos 0.5
    assert abs(tab[50, 3] - 0.479425538604203) < 1e-7         # sin 0.5
    tab = _table(200, 64, 1.0e6).astype(np.float64)
    c, s = tab[:, :32], tab[:, 32:]
    p, q = 37, 120
    assert np.abs(c[p + q] - (c[p] * c[q] - s[p] * s[q])).max() < 1e-6
    assert np.abs(s[p + q] - (s[p] * c[q] + c[p] * s[q])).max() < 1e-6
    assert np.abs(c * c + s * s - 1).max() < 1e-6
    # the slowest frequency: theta_{d/2-1} = base^(-(d-2)/d)
    assert abs(math.atan2(s[1, 31], c[1, 31]) - 1.0e6 ** (-62 / 64)) < 1e-9


def test_position_zero_without_norm_is_the_identity():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 64)).astype(np.float32)
    out = oracle.norm_rope(x, None, 1e-6, _table(8, 64), np.zeros(5, dtype=np.int64))
    assert np.array_equal(out, x.astype(np.float64))


def test_rope_is_a_complex_rotation_of_the_pairs_i_and_i_plus_half():
    """NeoX pairing: (x_i, x_{i+d/2}) rotates by pos * theta_i.  numpy's complex product is the
    independent routine; an interleaved (x_2i, x_2i+1) pairing or a flipped sign fails it."""
    rng = np.random.default_rng(2)
    T, H, d = 7, 2, 32
    x = rng.standard_normal((T, H, d)).astype(np.float32)
    pos = np.array([0, 1, 5, 17, 100, 511, 3])
    tab = _table(512, d)
    out = oracle.norm_rope(x, None, 0.0, tab, pos)
    z = x[..., : d // 2].astype(np.complex128) + 1j * x[..., d // 2:].astype(np.complex128)
    rot = (tab[pos, : d // 2].astype(np.float64) + 1j * tab[pos, d // 2:].astype(np.float64))[:, None, :]
    ref = z * rot
    assert np.abs(out[..., : d // 2] - ref.real).max() < 1e-12
    assert np.abs(out[..., d // 2:] - ref.imag).max() < 1e-12
    # a unit vector on axis 1 ends on axes 1 and 1 + d/2 only
    e = np.zeros((1, 1, d), dtype=np.float32)
    e[0, 0, 1] = 1.0
    o = oracle.norm_rope(e, None, 0.0, tab, np.array([9]))[0, 0]
    assert abs(o[1] - tab[9, 1]) < 1e-12 and abs(o[1 + d // 2] - tab[9, d // 2 + 1]) < 1e-12
    o[[1, 1 + d // 2]] = 0
    assert np.all(o == 0)


def test_rope_keeps_norms_and_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(3)
    d = 128
    q = rng.standard_normal((1, 1, d)).astype(np.float32)
    k = rng.standard_normal((1, 1, d)).astype(np.float32)
    tab = synth.make_rope_table(4096, d, 1.0e6).numpy()
    dots = []
    for shift in (0, 1, 777, 3000):
        qr = oracle.norm_rope(q, None, 0.0, tab, np.array([900 + shift]))
        kr = oracle.norm_rope(k, None, 0.0, tab, np.array([123 + shift]))
        assert abs(np.linalg.norm(qr) - np.linalg.norm(q.astype(np.float64))) < 1e-5
        dots.append(float((qr * kr).sum()))
    assert max(dots) - min(dots) < 2e-4      # the table is fp32: angles agree to ~1e-7 * position


def test_rmsnorm_closed_forms_and_library_routine():
    d = 64
    tab = _table(4, d)
    pos0 = np.zeros(1, dtype=np.int64)
    ones = np.ones(d, dtype=np.float32)
    # constant vector: y = c / sqrt(c^2 + eps)
    x = np.full((1, 1, d), 3.0, dtype=np.float32)
    y = oracle.norm_rope(x, ones, 0.25, tab, pos0)
    assert np.abs(y - 3.0 / math.sqrt(9.25)).max() < 1e-14
    # a 3-4-0... vector: mean square = 25/d
    x = np.zeros((1, 1, d), dtype=np.float32)
    x[0, 0, 0], x[0, 0, 40] = 3.0, 4.0
    y = oracle.norm_rope(x, ones, 0.0, tab, pos0)[0, 0]
    assert abs(y[0] - 3.0 / math.sqrt(25.0 / d)) < 1e-12 and abs(y[40] - 4.0 / math.sqrt(25.0 / d)) < 1e-12
    # eps = 0: scale invariant, unit mean square; the weight multiplies element-wise
    rng = np.random.default_rng(4)
    x = rng.standard_normal((6, 2, d)).astype(np.float32)
    w = (1 + 0.3 * rng.standard_normal(d)).astype(np.float32)
    p6 = np.zeros(6, dtype=np.int64)
    y1 = oracle.norm_rope(x, ones, 0.0, tab, p6)
    y2 = oracle.norm_rope(4.0 * x, ones, 0.0, tab, p6)
    assert np.abs(y1 - y2).max() < 1e-12
    assert np.abs((y1 ** 2).mean(-1) - 1).max() < 1e-12
    yw = oracle.norm_rope(x, w, 1e-6, tab, p6)
    assert np.abs(yw - oracle.norm_rope(x, ones, 1e-6, tab, p6) * w).max() < 1e-12
    # library routine in fp64
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (d,), torch.from_numpy(w).double(), 1e-6)
    assert np.abs(yw - ref.numpy()).max() < 1e-12


def test_norm_comes_before_the_rotation():
    """RMSNorm with a non-constant weight does not commute with the rotation; the step order is
    norm, then RoPE (weights applied to the unrotated vector)."""
    rng = np.random.default_rng(5)
    d = 32
    x = rng.standard_normal((1, 1, d)).astype(np.float32)
    w = (1 + 0.5 * rng.standard_normal(d)).astype(np.float32)
    tab = _table(64, d)
    pos = np.array([11])
    both = oracle.norm_rope(x, w, 1e-6, tab, pos)
    normed = oracle.norm_rope(x, w, 1e-6, tab, np.zeros(1, dtype=np.int64))       # norm only (pos 0)
    z = normed[0, 0, : d // 2] + 1j * normed[0, 0, d // 2:]
    rot = tab[11, : d // 2].astype(np.float64) + 1j * tab[11, d // 2:].astype(np.float64)
    assert np.abs(both[0, 0, : d // 2] - (z * rot).real).max() < 1e-6      # normed was rounded through fp64 only
    assert np.abs(both[0, 0, d // 2:] - (z * rot).imag).max() < 1e-6


def test_position_outside_the_table_is_refused():
    x = np.zeros((1, 1, 8), dtype=np.float32)
    with pytest.raises(AssertionError):
        oracle.norm_rope(x, None, 0.0, _table(4, 8), np.array([4]))


def test_f32_instantiation_stays_close():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((9, 3, 128)).astype(np.float32)
    w = (1 + 0.2 * rng.standard_normal(128)).astype(np.float32)
    tab = synth.make_rope_table(300, 128).numpy()
    pos = rng.integers(0, 300, 9)
    a = oracle.norm_rope(x, w, 1e-6, tab, pos)
    b = oracle.norm_rope(x, w, 1e-6, tab, pos, f32=True)
    assert np.abs(a - b).max() < 2e-5


def test_paged_scatter_places_position_p_in_page_p_div_ps_slot_p_mod_ps():
    rng = np.random.default_rng(7)
    ps, Hkv, d = 16, 2, 8
    bt = np.array([5, 2, 9, 0])
    cache = np.zeros((10, Hkv, ps, d), dtype=np.float32)
    rows = rng.standard_normal((20, Hkv, d)).astype(np.float32)
    pos = np.arange(30, 50)
    oracle.paged_scatter(rows, pos, bt, ps, cache)
    assert np.array_equal(cache[2, :, 14], rows[0]) and np.array_equal(cache[2, :, 15], rows[1])   # 30, 31 -> page 1
    assert np.array_equal(cache[9, :, 0], rows[2]) and np.array_equal(cache[0, :, 1], rows[19])    # 32 -> page 2; 49 -> page 3
    assert np.count_nonzero(cache) == rows.size
