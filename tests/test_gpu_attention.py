"""GPU parity: the three attention regimes against the CPU oracle (tolerance) and against
each other (zero differing bits), through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth
from gpu_common import ATTN_TOL, Rollout, bits, count_diff

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _oracle_packed(w, q, k, v):
    out, _ = oracle.attn_packed(q.float().cpu().numpy(), k.float().cpu().numpy(),
                                v.float().cpu().numpy(), w.cu_seqlens(), w.softmax_scale)
    return out


def _train(tik, w, q, k, v, cu, max_seqlen=None, lse=None):
    return tik.tik_attn_train_fwd(q, k, v, cu, max_seqlen or max(w.seq_lens), w.softmax_scale, lse=lse)


WORKLOADS = {
    "tiny": lambda: synth.get_workload(0),
    "d128_ragged": lambda: synth.custom_workload([100, 129, 1, 300], [57, 200, 3, 213], 8, 2, 128, 64),
    "d64_page32": lambda: synth.custom_workload([33, 250], [95, 140], 6, 3, 64, 32),
    "d128_page16_g1": lambda: synth.custom_workload([70], [186], 2, 2, 128, 16),
    "d128_page128_g16": lambda: synth.custom_workload([128, 5], [130, 250], 16, 1, 128, 128),
    "d64_page64_g32": lambda: synth.custom_workload([40, 130], [100, 30], 32, 1, 64, 64),
}


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_train_fwd_matches_oracle(tik, name):
    w = WORKLOADS[name]()
    q, k, v, cu = synth.make_qkv(w, "cuda")
    lse = torch.full((w.total_tokens, w.Hq), -1.0, dtype=torch.float32, device="cuda")
    o = _train(tik, w, q, k, v, cu, lse=lse)
    ref, ref_lse = oracle.attn_packed(q.float().cpu().numpy(), k.float().cpu().numpy(),
                                      v.float().cpu().numpy(), w.cu_seqlens(), w.softmax_scale)
    err = np.abs(o.float().cpu().numpy() - ref).max()
    assert err <= ATTN_TOL, err
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 1e-3
    # position 0 of every sequence attends one key: the output is that V row, bit for bit
    cu_h = w.cu_seqlens()
    for s in range(w.S):
        for h in range(w.Hq):
            assert torch.equal(bits(o[cu_h[s], h]), bits(v[cu_h[s], h // w.G]))


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_rollout_replay_is_bit_identical_to_train_fwd(tik, name):
    """Eq. 1: update-forward rows == prefill rows || decode rows, at every position."""
    w = WORKLOADS[name]()
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = _train(tik, w, q, k, v, cu)
    layout = synth.make_paged_layout(w)
    o_roll = Rollout(tik, w, q, k, v, layout).replay()
    assert count_diff(o_train, o_roll) == 0
    ref = _oracle_packed(w, q, k, v)
    assert np.abs(o_roll.float().cpu().numpy() - ref).max() <= ATTN_TOL


def test_multi_chunk_sequences(tik):
    """Contexts longer than one 2048-key chunk: in-kernel fold (train/prefill) and the
    split-KV combine (decode) agree bit for bit and with the oracle."""
    w = synth.custom_workload([2100, 1500], [2200, 700], 4, 2, 128, 64)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = _train(tik, w, q, k, v, cu)
    ref = _oracle_packed(w, q, k, v)
    assert np.abs(o_train.float().cpu().numpy() - ref).max() <= ATTN_TOL
    layout = synth.make_paged_layout(w)
    ro = Rollout(tik, w, q, k, v, layout)
    rows, o = ro.prefill()
    assert count_diff(o, o_train[rows]) == 0
    # fill the rest of the cache, then decode a few late positions directly
    cu_h = w.cu_seqlens()
    rest = [(s, w.prompt_lens[s], w.seq_lens[s]) for s in range(w.S)]
    rows2, o2 = ro.prefill(seqs=[r[0] for r in rest], start=[r[1] for r in rest], stop=[r[2] for r in rest])
    assert count_diff(o2, o_train[rows2]) == 0
    for pos in ([2047, 1499], [2048, 2047], [4299, 2199], [4096, 2048]):
        # K/V of those positions are already in the cache; rewriting them is idempotent
        rows3, o3 = ro.decode_step([0, 1], pos)
        assert count_diff(o3, o_train[rows3]) == 0, pos


def test_kv_cache_write_is_exact(tik):
    w = synth.get_workload(0)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    layout = synth.make_paged_layout(w)
    ro = Rollout(tik, w, q, k, v, layout, dirty=3.0)
    upto = [40, 64]
    ro.prefill(stop=upto)
    # expected pool: the oracle's index definition applied to a pool of the same dirty value
    # (bf16 -> fp32 is exact, so the comparison below is a bit comparison)
    shape = (layout.num_pages, w.Hkv, layout.page_size, w.d)
    kc_ref = np.full(shape, 3.0, dtype=np.float32)
    vc_ref = np.full(shape, 3.0, dtype=np.float32)
    cu_h = w.cu_seqlens()
    for s, n in enumerate(upto):
        sl = slice(int(cu_h[s]), int(cu_h[s]) + n)
        oracle.paged_scatter(k[sl].float().cpu().numpy(), np.arange(n), layout.block_table[s], layout.page_size, kc_ref)
        oracle.paged_scatter(v[sl].float().cpu().numpy(), np.arange(n), layout.block_table[s], layout.page_size, vc_ref)
    assert np.array_equal(ro.kc.float().cpu().numpy(), kc_ref) and np.array_equal(ro.vc.float().cpu().numpy(), vc_ref)
    assert (kc_ref != 3.0).any() and (kc_ref == 3.0).any()      # rows written and rows left alone both exist


def test_invalid_arguments_are_rejected(tik):
    w = synth.get_workload(0)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    k2 = torch.cat([k, k], 1).contiguous()
    with pytest.raises(tik.TikError):
        tik.tik_attn_train_fwd(q[:, :3].contiguous(), k2, k2, cu, 160, w.softmax_scale)    # Hq % Hkv
    with pytest.raises(tik.TikError):
        tik.tik_attn_train_fwd(q, k, v, cu, 160, -1.0)
    q96 = torch.zeros(4, 4, 96, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tik.TikError):
        tik.tik_attn_train_fwd(q96, q96[:, :1].contiguous(), q96[:, :1].contiguous(),
                               torch.tensor([0, 4], dtype=torch.int32, device="cuda"), 4, 0.1)
    layout = synth.make_paged_layout(w)
    kc, vc = synth.fill_paged_cache(w, layout, k, v)
    bt = torch.from_numpy(layout.block_table).cuda()
    ctx = torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda")
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(tik.TikError):
        tik.tik_attn_decode(q[:2].contiguous(), ctx, kc, vc, bt, 160, w.softmax_scale, ws=small)


def test_decode_context_above_the_host_bound_is_cut_and_flagged(tik):
    """ctx_lens[b] > max_ctx_len: the grid and the scratch were sized from the bound, so that slot
    is computed over keys 0..max_ctx_len-1 only, TIK_DEV_BAD_CONTEXT is raised, the other slots keep
    their bits and nothing is written beyond the scratch that the bound asks for."""
    w = synth.custom_workload([100, 100, 100], [2000, 4500, 1948], 8, 2, 128, 64)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros(layout.num_pages, w.Hkv, layout.page_size, w.d, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    tik.tik_kv_cache_write(k, v, cu, torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda"), kc, vc, bt)
    cu_h = w.cu_seqlens()
    bound = 2100                                              # two chunks; sequence 1 holds 4600 keys
    qd = torch.stack([q[int(cu_h[0]) + 2099], q[int(cu_h[1]) + 2099], q[int(cu_h[2]) + 2047]]).contiguous()
    good = torch.tensor([2100, 2100, 2048], dtype=torch.int32, device="cuda")
    ref = tik.tik_attn_decode(qd, good, kc, vc, bt, bound, w.softmax_scale)
    assert tik.device_status() == 0
    need = tik.workspace_bytes(tik.OP_ATTN_DECODE, 3, w.Hq, w.Hkv, w.d, bound)
    ws = torch.full((need + 4096,), 0x5A, dtype=torch.uint8, device="cuda")
    bad = torch.tensor([2100, 4600, 2048], dtype=torch.int32, device="cuda")     # 3 chunks claimed, 2 allowed
    out = tik.tik_attn_decode(qd, bad, kc, vc, bt, bound, w.softmax_scale, ws=ws)
    flags = tik.device_status()
    assert flags == tik.DEV_BAD_CONTEXT
    assert count_diff(out, ref) == 0                          # slot 1 cut to the bound, slots 0 and 2 untouched by it
    assert bool((ws[need:] == 0x5A).all())


def test_prefill_kv_equals_cache_write_then_prefill(tik):
    """The one-call form leaves the same cache and the same output bits as the two calls, also for a
    second chunk behind a cached prefix."""
    w = synth.custom_workload([300, 1100, 64], [1, 1, 1], 8, 2, 128, 64)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    layout = synth.make_paged_layout(w)
    ro = Rollout(tik, w, q, k, v, layout)
    cu_h = w.cu_seqlens()
    kc = torch.zeros_like(ro.kc)
    vc = torch.zeros_like(ro.vc)
    for a, b in (([0, 0, 0], [170, 1000, 64]), ([170, 1000, 64], [300, 1100, 64])):
        rows, o_ref = ro.prefill(start=a, stop=b)
        lens = [y - x for x, y in zip(a, b)]
        if max(lens) == 0:
            continue
        cu_q = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
        ctx = torch.tensor(b, dtype=torch.int32, device="cuda")
        o = tik.tik_attn_prefill_kv(q[rows].contiguous(), k[rows].contiguous(), v[rows].contiguous(), cu_q, ctx, kc, vc,
                                    ro.bt, max(lens), max(b), w.softmax_scale)
        assert count_diff(o, o_ref) == 0
        assert torch.equal(bits(kc), bits(ro.kc)) and torch.equal(bits(vc), bits(ro.vc))
