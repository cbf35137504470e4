"""GPU parity of the pre-attention step (per-head RMSNorm -> NeoX RoPE -> indexed cache write)
against the CPU oracle, and its bit-identity between the full-sequence call of the policy update
and the prompt / token-wise calls of the rollout (the paper's operator table verifies these
operators bitwise between the two uses, cache post-write state included)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth
from gpu_common import bits, count_diff

pytestmark = pytest.mark.gpu

EPS = 1e-6
CASES = {
    "d128_g4": lambda: synth.custom_workload([100, 129, 1, 300], [57, 200, 3, 213], 8, 2, 128, 64, index=40),
    "d64_g2": lambda: synth.custom_workload([33, 250], [95, 140], 6, 3, 64, 32, index=41),
    "d128_heads40": lambda: synth.custom_workload([70, 5], [186, 60], 32, 8, 128, 16, index=42),
}


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _positions(w):
    return np.concatenate([np.arange(L) for L in w.seq_lens])


def _check_against_oracle(got, x, wt, tab, pos):
    ref = oracle.norm_rope(x.float().cpu().numpy(), None if wt is None else wt.float().cpu().numpy(), EPS,
                           tab.cpu().numpy(), pos)
    g = got.float().cpu().numpy().astype(np.float64)
    # one bf16 rounding (relative 2^-9) on top of fp32 arithmetic
    assert np.all(np.abs(g - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-6)
    rounded = torch.from_numpy(ref).to(torch.bfloat16).float().numpy()
    assert np.mean(rounded != g) < 0.01       # almost every element is the correctly rounded oracle value


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("with_norm", [True, False])
def test_full_sequence_call_matches_oracle(tik, name, with_norm):
    w = CASES[name]()
    q0, k0, v, cu = synth.make_qkv(w, "cuda")
    wq, wk = synth.make_norm_weights(w, "cuda") if with_norm else (None, None)
    tab = synth.make_rope_table(max(w.seq_lens) + 7, w.d, device="cuda")
    q, k = q0.clone(), k0.clone()
    tik.tik_qk_norm_rope_kv_write(q, k, None, wq, wk, EPS, tab, cu)
    pos = _positions(w)
    _check_against_oracle(q, q0, wq, tab, pos)
    _check_against_oracle(k, k0, wk, tab, pos)
    # position 0 without norm is the identity, bit for bit
    if not with_norm:
        first = torch.from_numpy(w.cu_seqlens()[:-1].astype(np.int64)).cuda()
        assert count_diff(q[first], q0[first]) == 0 and count_diff(k[first], k0[first]) == 0


@pytest.mark.parametrize("name", list(CASES))
def test_rollout_calls_give_the_bits_of_the_full_sequence_call(tik, name):
    w = CASES[name]()
    q0, k0, v, cu = synth.make_qkv(w, "cuda")
    wq, wk = synth.make_norm_weights(w, "cuda")
    tab = synth.make_rope_table(max(w.seq_lens), w.d, device="cuda")
    q_full, k_full = q0.clone(), k0.clone()
    tik.tik_qk_norm_rope_kv_write(q_full, k_full, None, wq, wk, EPS, tab, cu)

    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    shape = (layout.num_pages, w.Hkv, layout.page_size, w.d)
    kc = torch.full(shape, -7.0, dtype=torch.bfloat16, device="cuda")
    vc = torch.full(shape, -7.0, dtype=torch.bfloat16, device="cuda")
    cu_h = w.cu_seqlens()
    q_roll, k_roll = torch.empty_like(q0), torch.empty_like(k0)
    # prompts in one call
    rows = torch.cat([torch.arange(cu_h[s], cu_h[s] + w.prompt_lens[s]) for s in range(w.S)]).cuda()
    cu_p = torch.tensor(np.concatenate([[0], np.cumsum(w.prompt_lens)]), dtype=torch.int32, device="cuda")
    qp, kp, vp = q0[rows].contiguous(), k0[rows].contiguous(), v[rows].contiguous()
    tik.tik_qk_norm_rope_kv_write(qp, kp, vp, wq, wk, EPS, tab, cu_p,
                                  torch.tensor(w.prompt_lens, dtype=torch.int32, device="cuda"), kc, vc, bt)
    q_roll[rows], k_roll[rows] = qp, kp
    # responses one token per live sequence per call
    for t in range(max(w.response_lens)):
        live = [s for s in range(w.S) if t < w.response_lens[s]]
        r = torch.tensor([int(cu_h[s]) + w.prompt_lens[s] + t for s in live], device="cuda")
        qd, kd, vd = q0[r].contiguous(), k0[r].contiguous(), v[r].contiguous()
        ctx = torch.tensor([w.prompt_lens[s] + t + 1 for s in live], dtype=torch.int32, device="cuda")
        cu_d = torch.arange(len(live) + 1, dtype=torch.int32, device="cuda")
        tik.tik_qk_norm_rope_kv_write(qd, kd, vd, wq, wk, EPS, tab, cu_d, ctx, kc, vc, bt[live].contiguous())
        q_roll[r], k_roll[r] = qd, kd
    assert count_diff(q_roll, q_full) == 0
    assert count_diff(k_roll, k_full) == 0
    # cache post-write state: the index definition applied to the transformed K and to V
    kc_ref = np.full(shape, -7.0, dtype=np.float32)
    vc_ref = np.full(shape, -7.0, dtype=np.float32)
    kf, vf = k_full.float().cpu().numpy(), v.float().cpu().numpy()
    for s in range(w.S):
        sl = slice(int(cu_h[s]), int(cu_h[s + 1]))
        oracle.paged_scatter(kf[sl], np.arange(w.seq_lens[s]), layout.block_table[s], layout.page_size, kc_ref)
        oracle.paged_scatter(vf[sl], np.arange(w.seq_lens[s]), layout.block_table[s], layout.page_size, vc_ref)
    assert np.array_equal(kc.float().cpu().numpy(), kc_ref)
    assert np.array_equal(vc.float().cpu().numpy(), vc_ref)


def test_prepared_rollout_attention_equals_prepared_train_forward(tik):
    """raw q, k, v -> pre-attention step -> attention, through both regimes, end to end."""
    w = CASES["d128_g4"]()
    q0, k0, v, cu = synth.make_qkv(w, "cuda")
    wq, wk = synth.make_norm_weights(w, "cuda")
    tab = synth.make_rope_table(max(w.seq_lens), w.d, device="cuda")
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros(layout.num_pages, w.Hkv, layout.page_size, w.d, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    q, k = q0.clone(), k0.clone()
    ctx = torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda")
    tik.tik_qk_norm_rope_kv_write(q, k, v, wq, wk, EPS, tab, cu, ctx, kc, vc, bt)
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale)
    o_pre = tik.tik_attn_prefill(q, cu, ctx, kc, vc, bt, max(w.seq_lens), max(w.seq_lens), w.softmax_scale)
    assert count_diff(o_pre, o_train) == 0
    cu_h = w.cu_seqlens()
    last = torch.tensor([int(cu_h[s + 1]) - 1 for s in range(w.S)], device="cuda")
    o_dec = tik.tik_attn_decode(q[last].contiguous(), ctx, kc, vc, bt, max(w.seq_lens), w.softmax_scale)
    assert count_diff(o_dec, o_train[last]) == 0
    ref, _ = oracle.attn_packed(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(),
                                cu_h, w.softmax_scale)
    assert np.abs(o_train.float().cpu().numpy() - ref).max() <= 2e-2


def test_bad_position_and_bad_block_are_flagged_and_skipped(tik):
    w = synth.custom_workload([10], [10], 4, 2, 64, 16, index=43)
    q0, k0, v, cu = synth.make_qkv(w, "cuda")
    tab = synth.make_rope_table(12, w.d, device="cuda")          # positions 12..19 have no table row
    q, k = q0.clone(), k0.clone()
    tik.tik_qk_norm_rope_kv_write(q, k, None, None, None, EPS, tab, cu)
    assert tik.device_status() == tik.DEV_BAD_POSITION
    assert count_diff(q[12:], q0[12:]) == 0 and count_diff(k[12:], k0[12:]) == 0
    assert count_diff(q[1:12], q0[1:12]) > 0
    # a block-table entry out of range: q and k are still transformed, nothing lands in the cache
    tab = synth.make_rope_table(32, w.d, device="cuda")
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    bt[0, 1] = layout.num_pages + 5
    kc = torch.full((layout.num_pages, w.Hkv, 16, w.d), 3.0, dtype=torch.bfloat16, device="cuda")
    vc = torch.full_like(kc, 3.0)
    q2, k2 = q0.clone(), k0.clone()
    ctx = torch.tensor([20], dtype=torch.int32, device="cuda")
    tik.tik_qk_norm_rope_kv_write(q2, k2, v, None, None, EPS, tab, cu, ctx, kc, vc, bt)
    assert tik.device_status() == tik.DEV_BAD_BLOCK
    good = torch.ones(layout.num_pages, dtype=torch.bool)
    good[int(bt[0, 0])] = False
    assert bool((kc[good.cuda()] == 3.0).all())              # only page 0 of the sequence was written
    assert count_diff(kc[int(bt[0, 0])].transpose(0, 1)[:16], k2[:16]) == 0
    # empty call and argument errors
    tik.tik_qk_norm_rope_kv_write(q0[:0], k0[:0], None, None, None, EPS, tab,
                                  torch.zeros(1, dtype=torch.int32, device="cuda"))
    with pytest.raises(tik.TikError):
        tik.tik_qk_norm_rope_kv_write(q0.clone(), k0.clone(), None, None, None, float("nan"), tab, cu)
    with pytest.raises(tik.TikError):        # a cache without V
        tik.tik_qk_norm_rope_kv_write(q0.clone(), k0.clone(), None, None, None, EPS, tab, cu, ctx, kc, vc, bt)
