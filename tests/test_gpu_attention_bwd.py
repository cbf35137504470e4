"""GPU parity of the attention backward (policy-update backward) against the CPU oracle, its
run-to-run determinism and its independence of batch composition."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth
from gpu_common import count_diff

pytestmark = pytest.mark.gpu

# bf16 weights and score gradients feed the tensor cores and the results are rounded to bf16 once:
# errors are a few 2^-9 of the tensor's scale
BWD_MAX_REL = 2e-2       # max |got - ref| / max |ref|
BWD_RMS_REL = 6e-3       # rms(got - ref) / rms(ref)

CASES = {
    "d128_ragged": lambda: synth.custom_workload([100, 129, 1, 300], [57, 200, 3, 213], 8, 2, 128, 64, index=50),
    "d64_g2": lambda: synth.custom_workload([33, 250], [95, 140], 6, 3, 64, 32, index=51),
    "d128_g1_long": lambda: synth.custom_workload([700], [600], 2, 2, 128, 64, index=52),
    "d128_g16_tiny": lambda: synth.custom_workload([1, 5], [0, 130], 16, 1, 128, 64, index=53),
    # 21 tiles: the K / V rings of the dQ pass and the stage ring of the dK/dV pass wrap many times
    "d128_g2_rings": lambda: synth.custom_workload([1300], [1300], 2, 1, 128, 64, index=54),
    # head_dim 64 over 18 tiles, and a grouped-query sequence longer than one 2048-key chunk
    "d64_g2_18tiles": lambda: synth.custom_workload([1100], [1150], 4, 2, 64, 32, index=55),
    "d128_g4_multichunk": lambda: synth.custom_workload([900, 40], [1700, 9], 4, 1, 128, 64, index=56),
}


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _fwd_bwd(tik, w, q, k, v, cu, do):
    lse = torch.empty(q.shape[0], w.Hq, dtype=torch.float32, device="cuda")
    o = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale, lse=lse)
    return tik.tik_attn_train_bwd(q, k, v, o, do, lse, cu, max(w.seq_lens), w.softmax_scale)


def _check(got, ref, name):
    g = got.float().cpu().numpy().astype(np.float64)
    err = g - ref
    assert np.abs(err).max() <= BWD_MAX_REL * np.abs(ref).max(), (name, np.abs(err).max(), np.abs(ref).max())
    assert np.sqrt((err ** 2).mean()) <= BWD_RMS_REL * np.sqrt((ref ** 2).mean()), name


@pytest.mark.parametrize("name", list(CASES))
def test_backward_matches_oracle_and_is_deterministic(tik, name):
    w = CASES[name]()
    q, k, v, cu = synth.make_qkv(w, "cuda")
    do, _, _, _ = synth.make_qkv(w, "cuda", seed_offset=9)
    dq, dk, dv = _fwd_bwd(tik, w, q, k, v, cu, do)
    rq, rk, rv = oracle.attn_bwd_packed(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(),
                                        do.float().cpu().numpy(), w.cu_seqlens(), w.softmax_scale)
    _check(dq, rq, "dq")
    _check(dk, rk, "dk")
    _check(dv, rv, "dv")
    assert bool(torch.isfinite(dq).all() and torch.isfinite(dk).all() and torch.isfinite(dv).all())
    # same inputs, same bits
    dq2, dk2, dv2 = _fwd_bwd(tik, w, q, k, v, cu, do)
    assert count_diff(dq, dq2) == 0 and count_diff(dk, dk2) == 0 and count_diff(dv, dv2) == 0
    # position 0 of every sequence: softmax over one key is constant, no gradient reaches q_0
    # (up to the rounding of o, which enters delta)
    first = torch.from_numpy(w.cu_seqlens()[:-1].astype(np.int64)).cuda()
    assert float(dq[first].float().abs().max()) <= 1e-2 * float(np.abs(rq).max())


def test_backward_does_not_depend_on_batch_composition(tik):
    w = CASES["d128_ragged"]()
    q, k, v, cu = synth.make_qkv(w, "cuda")
    do, _, _, _ = synth.make_qkv(w, "cuda", seed_offset=9)
    dq, dk, dv = _fwd_bwd(tik, w, q, k, v, cu, do)
    cu_h = w.cu_seqlens()
    for s in (1, 3):
        sl = slice(int(cu_h[s]), int(cu_h[s + 1]))
        w1 = synth.custom_workload([w.prompt_lens[s]], [w.response_lens[s]], w.Hq, w.Hkv, w.d, 64)
        cu1 = torch.tensor([0, w.seq_lens[s]], dtype=torch.int32, device="cuda")
        dq1, dk1, dv1 = _fwd_bwd(tik, w1, q[sl].contiguous(), k[sl].contiguous(), v[sl].contiguous(), cu1,
                                 do[sl].contiguous())
        assert count_diff(dq1, dq[sl]) == 0 and count_diff(dk1, dk[sl]) == 0 and count_diff(dv1, dv[sl]) == 0


def test_backward_invalid_arguments(tik):
    w = CASES["d64_g2"]()
    q, k, v, cu = synth.make_qkv(w, "cuda")
    lse = torch.zeros(q.shape[0], w.Hq, dtype=torch.float32, device="cuda")
    with pytest.raises(tik.TikError):
        tik.tik_attn_train_bwd(q, k, v, q, q, lse, cu, max(w.seq_lens), w.softmax_scale,
                               ws=torch.empty(16, dtype=torch.uint8, device="cuda"))
