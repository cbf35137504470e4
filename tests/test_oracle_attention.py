"""Pins for the CPU attention oracle: closed forms, invariants, brute force and a
library cross-check.  None of these re-use the oracle's own code path to make
the expected value."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16).float().numpy()


def _tiny_inputs():
    w = synth.get_workload(0)
    q, k, v, cu = synth.make_qkv(w)
    return w, q.float().numpy(), k.float().numpy(), v.float().numpy(), cu.numpy()


# --------------------------------------------------------------------------- golden
def _parse_attn_golden():
    cases = []
    with open(os.path.join(GOLDEN, "attn_closed_form.txt")) as f:
        for line in f:
            if not line.startswith("case"):
                continue
            parts = [p.split() for p in line[4:].split("|")]
            scale, qscale = float(parts[0][0]), float(parts[0][1])
            w = [int(x) for x in parts[1]]
            a = [float(x) for x in parts[2]]
            b = [float(x) for x in parts[3]]
            t = int(parts[4][0])
            exp = [Fraction(x) for x in parts[5]]
            cases.append((scale, qscale, w, a, b, t, exp))
    return cases


@pytest.mark.parametrize("case", _parse_attn_golden())
def test_golden_rational_weights(case):
    scale, qscale, w, a, b, t, exp = case
    n = len(w)
    L = n
    q = np.zeros((L, 1, 2), np.float32)
    q[:, 0, 0] = qscale
    k = np.zeros((L, 1, 2), np.float32)
    k[:, 0, 0] = [math.log(x) / (scale * qscale) for x in w]
    k[:, 0, 1] = np.arange(L) * 3.0 - 1.0        # ignored: q's second coordinate is 0
    v = np.stack([np.array(a, np.float32), np.array(b, np.float32)], -1).reshape(L, 1, 2)
    out, lse = oracle.attn_packed(q, k, v, [0, L], scale)
    got = out[t, 0]
    for c in range(2):
        assert abs(got[c] - float(exp[c])) < 2e-6, (got, exp)
    # lse of the row is ln(sum of the weights) by the same construction
    assert abs(lse[t, 0] - math.log(sum(w[: t + 1]))) < 2e-6


# --------------------------------------------------------------------------- invariants
def test_softmax_rows_sum_to_one():
    w, q, k, v, cu = _tiny_inputs()
    for s in range(w.S):
        for t in (0, 1, 63, 64, w.seq_lens[s] - 1):
            row = cu[s] + t
            probs, out = oracle.attn_probs(q[row, 2], k[cu[s]:row + 1, 0], v[cu[s]:row + 1, 0],
                                           w.softmax_scale)
            assert probs.shape == (t + 1,)
            assert abs(probs.sum() - 1.0) < 1e-12
            assert (probs >= 0).all()
            np.testing.assert_allclose(out, probs @ v[cu[s]:row + 1, 0].astype(np.float64),
                                       atol=1e-12)


def test_identical_keys_give_running_mean_of_v():
    L, Hq, Hkv, d = 70, 4, 2, 16
    q = _rand((L, Hq, d), 1)
    k = np.broadcast_to(_rand((1, Hkv, d), 2), (L, Hkv, d)).copy()
    v = _rand((L, Hkv, d), 3)
    out, lse = oracle.attn_packed(q, k, v, [0, L], 0.25)
    cum = np.cumsum(v.astype(np.float64), axis=0) / np.arange(1, L + 1)[:, None, None]
    for h in range(Hq):
        np.testing.assert_allclose(out[:, h], cum[:, h // 2], atol=1e-12)


def test_first_position_returns_v0_exactly():
    w, q, k, v, cu = _tiny_inputs()
    out, _ = oracle.attn_packed(q, k, v, cu, w.softmax_scale)
    for s in range(w.S):
        for h in range(w.Hq):
            assert np.array_equal(out[cu[s], h], v[cu[s], h // w.G].astype(np.float64))


def test_dominant_key_selects_its_value():
    L, d = 33, 8
    q = _rand((L, 1, d), 4)
    k = np.zeros((L, 1, d), np.float32)
    v = _rand((L, 1, d), 5)
    jstar = 11
    t = L - 1
    qhat = q[t, 0] / np.linalg.norm(q[t, 0])
    k[jstar, 0] = 60.0 * qhat
    out, _ = oracle.attn_packed(q, k, v, [0, L], 1.0)
    assert np.abs(out[t, 0] - v[jstar, 0]).max() < 1e-4 * max(1.0, np.abs(v).max())


def test_causality_future_tokens_do_not_matter():
    w, q, k, v, cu = _tiny_inputs()
    base, _ = oracle.attn_packed(q, k, v, cu, w.softmax_scale)
    t = 50
    k2, v2 = k.copy(), v.copy()
    for s in range(w.S):
        k2[cu[s] + t + 1:cu[s + 1]] += 3.0
        v2[cu[s] + t + 1:cu[s + 1]] -= 5.0
    pert, _ = oracle.attn_packed(q, k2, v2, cu, w.softmax_scale)
    for s in range(w.S):
        assert np.array_equal(base[cu[s]:cu[s] + t + 1], pert[cu[s]:cu[s] + t + 1])
        assert not np.array_equal(base[cu[s] + t + 1:cu[s + 1]], pert[cu[s] + t + 1:cu[s + 1]])


def test_sequences_are_independent():
    w, q, k, v, cu = _tiny_inputs()
    both, _ = oracle.attn_packed(q, k, v, cu, w.softmax_scale)
    for s in range(w.S):
        sl = slice(cu[s], cu[s + 1])
        alone, _ = oracle.attn_packed(q[sl], k[sl], v[sl], [0, cu[s + 1] - cu[s]],
                                      w.softmax_scale)
        assert np.array_equal(both[sl], alone)


def test_gqa_equals_mha_with_repeated_kv():
    L, Hq, Hkv, d = 40, 6, 2, 16
    q, k, v = _rand((L, Hq, d), 6), _rand((L, Hkv, d), 7), _rand((L, Hkv, d), 8)
    a, la = oracle.attn_packed(q, k, v, [0, 17, L], 0.3)
    G = Hq // Hkv
    b, lb = oracle.attn_packed(q, np.repeat(k, G, axis=1), np.repeat(v, G, axis=1), [0, 17, L],
                               0.3)
    assert np.array_equal(a, b) and np.array_equal(la, lb)


def test_key_shift_invariance():
    L, d = 48, 16
    q, k, v = _rand((L, 2, d), 9), _rand((L, 1, d), 10), _rand((L, 1, d), 11)
    a, _ = oracle.attn_packed(q, k, v, [0, L], 0.25)
    shift = _rand((1, 1, d), 12)
    b, _ = oracle.attn_packed(q, k + shift, v, [0, L], 0.25)
    assert np.abs(a - b).max() < 1e-4


def test_value_linearity():
    """Output is linear in V: attn(q,k,2v1+v2) = 2 attn(q,k,v1) + attn(q,k,v2)."""
    L, d = 24, 8
    q, k = _rand((L, 2, d), 13), _rand((L, 2, d), 14)
    v1, v2 = _rand((L, 2, d), 15), _rand((L, 2, d), 16)
    a, _ = oracle.attn_packed(q, k, v1, [0, L], 0.5)
    b, _ = oracle.attn_packed(q, k, v2, [0, L], 0.5)
    c, _ = oracle.attn_packed(q, k, 2 * v1 + v2, [0, L], 0.5)
    np.testing.assert_allclose(c, 2 * a + b, atol=1e-12)


# --------------------------------------------------------------------------- brute force
def _brute(q, k, v, cu, scale):
    tot, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    out = np.zeros((tot, Hq, d))
    lse = np.zeros((tot, Hq))
    for s in range(len(cu) - 1):
        for t in range(cu[s], cu[s + 1]):
            for h in range(Hq):
                g = h // G
                sc = []
                for j in range(cu[s], t + 1):
                    dot = 0.0
                    for c in range(d):
                        dot += float(q[t, h, c]) * float(k[j, g, c])
                    sc.append(scale * dot)
                den = sum(math.exp(x) for x in sc)
                for c in range(d):
                    out[t, h, c] = sum(math.exp(x) * float(v[cu[s] + i, g, c])
                                       for i, x in enumerate(sc)) / den
                lse[t, h] = math.log(den)
    return out, lse


def test_brute_force_tiny():
    Hq, Hkv, d = 4, 2, 4
    cu = [0, 5, 5, 13]          # includes an empty sequence
    q, k, v = _rand((13, Hq, d), 17), _rand((13, Hkv, d), 18), _rand((13, Hkv, d), 19)
    out, lse = oracle.attn_packed(q, k, v, cu, 0.7)
    bo, bl = _brute(q, k, v, cu, 0.7)
    np.testing.assert_allclose(out, bo, atol=1e-12)
    np.testing.assert_allclose(lse, bl, atol=1e-12)


# --------------------------------------------------------------------------- library cross-check
def test_matches_library_attention():
    L, Hq, Hkv, d = 96, 4, 2, 32
    q, k, v = _rand((L, Hq, d), 20), _rand((L, Hkv, d), 21), _rand((L, Hkv, d), 22)
    out, _ = oracle.attn_packed(q, k, v, [0, L], 1.0 / math.sqrt(d))
    tq = torch.from_numpy(q).double().permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.repeat(k, 2, axis=1)).double().permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(v, 2, axis=1)).double().permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    ref = ref[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(out, ref, atol=1e-10)


# --------------------------------------------------------------------------- entry points agree
def test_paged_equals_packed_and_rows_entry():
    w, q, k, v, cu = _tiny_inputs()
    packed, lse_p = oracle.attn_packed(q, k, v, cu, w.softmax_scale)
    for page in (16, 64):
        layout = synth.make_paged_layout(w, page_size=page)
        qt, kt, vt, _ = synth.make_qkv(w)
        kc, vc = synth.fill_paged_cache(w, layout, kt, vt)
        # whole sequences as one "prefill" against a full cache
        paged, lse_g = oracle.attn_paged(q, cu, w.seq_lens, kc.float().numpy(),
                                         vc.float().numpy(), layout.block_table,
                                         w.softmax_scale)
        assert np.array_equal(packed, paged) and np.array_equal(lse_p, lse_g)
        # decode-shaped: the last token of every sequence only
        last = np.array([cu[s + 1] - 1 for s in range(w.S)])
        dec, _ = oracle.attn_paged(q[last], np.arange(w.S + 1), w.seq_lens,
                                   kc.float().numpy(), vc.float().numpy(),
                                   layout.block_table, w.softmax_scale)
        assert np.array_equal(dec, packed[last])
    # sampled-rows entry
    rows = synth.sample_rows(w, 20)
    g = [h // w.G for (_, h, _) in rows]
    assert set(g) == {0}
    kflat, vflat = k[:, 0], v[:, 0]
    qr = np.stack([q[cu[s] + t, h] for (s, h, t) in rows])
    out, _ = oracle.attn_rows(qr, kflat, vflat, [cu[s] for (s, _, _) in rows],
                              [t + 1 for (_, _, t) in rows], w.softmax_scale)
    exp = np.stack([packed[cu[s] + t, h] for (s, h, t) in rows])
    assert np.array_equal(out, exp)


def test_paged_prefill_behind_cached_prefix():
    """Queries that start at a non-zero position attend the cached prefix too."""
    w, q, k, v, cu = _tiny_inputs()
    packed, _ = oracle.attn_packed(q, k, v, cu, w.softmax_scale)
    layout = synth.make_paged_layout(w)
    qt, kt, vt, _ = synth.make_qkv(w)
    kc, vc = synth.fill_paged_cache(w, layout, kt, vt)
    start = [37, 64]
    idx = np.concatenate([np.arange(cu[s] + start[s], cu[s + 1]) for s in range(w.S)])
    cuq = np.concatenate([[0], np.cumsum([w.seq_lens[s] - start[s] for s in range(w.S)])])
    out, _ = oracle.attn_paged(q[idx], cuq, w.seq_lens, kc.float().numpy(), vc.float().numpy(),
                               layout.block_table, w.softmax_scale)
    assert np.array_equal(out, packed[idx])


def test_fp32_arithmetic_variant_is_close():
    w, q, k, v, cu = _tiny_inputs()
    a, la = oracle.attn_packed(q, k, v, cu, w.softmax_scale)
    b, lb = oracle.attn_packed(q, k, v, cu, w.softmax_scale, f32=True)
    assert np.abs(a - b).max() < 1e-4
    assert np.abs(la - lb).max() < 1e-4
