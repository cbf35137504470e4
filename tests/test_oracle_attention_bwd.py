"""Pins for the attention-backward oracle: torch autograd through fp64 scaled_dot_product_attention
(a library routine), central finite differences of the forward oracle, and invariants that a dropped
term, a wrong sign or a transposed operand would break."""
import numpy as np
import torch

import oracle


def _inputs(seed, lens, Hq, Hkv, d):
    rng = np.random.default_rng(seed)
    tot = sum(lens)
    q = rng.standard_normal((tot, Hq, d)).astype(np.float32)
    k = rng.standard_normal((tot, Hkv, d)).astype(np.float32)
    v = rng.standard_normal((tot, Hkv, d)).astype(np.float32)
    do = rng.standard_normal((tot, Hq, d)).astype(np.float32)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    return q, k, v, do, cu


def test_against_torch_autograd_in_fp64():
    lens, Hq, Hkv, d = [5, 1, 9], 4, 2, 8
    q, k, v, do, cu = _inputs(21, lens, Hq, Hkv, d)
    scale = 0.3
    dq, dk, dv = oracle.attn_bwd_packed(q, k, v, do, cu, scale)
    G = Hq // Hkv
    for s in range(len(lens)):
        sl = slice(int(cu[s]), int(cu[s + 1]))
        tq = torch.from_numpy(q[sl]).double().permute(1, 0, 2).requires_grad_(True)
        tk = torch.from_numpy(k[sl]).double().permute(1, 0, 2).requires_grad_(True)
        tv = torch.from_numpy(v[sl]).double().permute(1, 0, 2).requires_grad_(True)
        out = torch.nn.functional.scaled_dot_product_attention(
            tq, tk.repeat_interleave(G, 0), tv.repeat_interleave(G, 0), is_causal=True, scale=scale)
        out.backward(torch.from_numpy(do[sl]).double().permute(1, 0, 2))
        assert np.abs(dq[sl] - tq.grad.permute(1, 0, 2).numpy()).max() < 1e-12
        assert np.abs(dk[sl] - tk.grad.permute(1, 0, 2).numpy()).max() < 1e-12
        assert np.abs(dv[sl] - tv.grad.permute(1, 0, 2).numpy()).max() < 1e-12


def test_against_finite_differences_of_the_forward_oracle():
    lens, Hq, Hkv, d = [4, 3], 2, 1, 4
    q, k, v, do, cu = _inputs(22, lens, Hq, Hkv, d)
    scale = 0.5
    dq, dk, dv = oracle.attn_bwd_packed(q, k, v, do, cu, scale)

    def loss(q_, k_, v_):
        out, _ = oracle.attn_packed(q_, k_, v_, cu, scale)
        return float((out * do).sum())

    rng = np.random.default_rng(0)
    h = 2.0 ** -7                     # exactly representable steps keep the fp32 inputs exact
    for arr, grad, idx in ((q, dq, 0), (k, dk, 1), (v, dv, 2)):
        for _ in range(6):
            pos = tuple(int(rng.integers(0, n)) for n in arr.shape)
            args = [q.copy(), k.copy(), v.copy()]
            args[idx][pos] += h
            up = loss(*args)
            args[idx][pos] -= 2 * h
            dn = loss(*args)
            assert abs((up - dn) / (2 * h) - grad[pos]) < 2e-4, (idx, pos)


def test_invariants():
    lens, Hq, Hkv, d = [6, 2], 2, 2, 4
    q, k, v, do, cu = _inputs(23, lens, Hq, Hkv, d)
    scale = 0.7
    dq, dk, dv = oracle.attn_bwd_packed(q, k, v, do, cu, scale)
    # position 0 attends only itself: softmax is constant 1, so no gradient reaches q_0; its dO goes to v_0
    for s in range(2):
        assert np.all(dq[cu[s]] == 0)
    # single-token sequence: dv = dO summed over the group's heads (one head per group here), dk = 0
    q1, k1, v1, do1, cu1 = _inputs(24, [1], 4, 2, 4)
    dq1, dk1, dv1 = oracle.attn_bwd_packed(q1, k1, v1, do1, cu1, scale)
    assert np.all(dk1 == 0) and np.all(dq1 == 0)
    assert np.abs(dv1[0, 0] - (do1[0, 0].astype(np.float64) + do1[0, 1])).max() < 1e-15
    assert np.abs(dv1[0, 1] - (do1[0, 2].astype(np.float64) + do1[0, 3])).max() < 1e-15
    # the sum of dv over keys equals the sum of dO over queries (softmax rows sum to one)
    assert np.abs(dv[: lens[0]].sum(0) - do[: lens[0]].astype(np.float64).sum(0)).max() < 1e-12
    # every row of dS sums to zero (softmax Jacobian), so sum_j dk_j = scale * sum_i (sum_j ds_ij) q_i = 0
    assert np.abs(dk[: lens[0]].sum(0)).max() < 1e-12
    # linear in dO; sequences independent
    dq2, dk2, dv2 = oracle.attn_bwd_packed(q, k, v, 2 * do, cu, scale)
    assert np.array_equal(dq2, 2 * dq) and np.array_equal(dk2, 2 * dk) and np.array_equal(dv2, 2 * dv)
    a = slice(int(cu[1]), int(cu[2]))
    dqs, dks, dvs = oracle.attn_bwd_packed(q[a], k[a], v[a], do[a], np.array([0, lens[1]], dtype=np.int32), scale)
    assert np.array_equal(dqs, dq[a]) and np.array_equal(dks, dk[a]) and np.array_equal(dvs, dv[a])
