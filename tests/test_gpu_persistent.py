"""The persistent schedule of the full-sequence kernels (a CTA walks a device-built list of work
items) against the one-CTA-per-item schedule: a schedule change must not move a bit (the paper's
bitwise-preservation check, Sec. 5.3), on length mixes that make a CTA cross every kind of item
boundary (pair -> pair, pair -> single tile, single -> pair, multi-chunk rows, ragged tiles)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35140_b200 import synth
from gpu_common import ATTN_TOL, count_diff

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _lens(seed, n, lo, hi):
    return [int(x) for x in np.random.default_rng(seed).integers(lo, hi + 1, n)]


CASES = {
    # many short sequences: every CTA walks several paired items
    "short_many": lambda: synth.custom_workload([1] * 96, _lens(1, 96, 1, 700), 8, 2, 128, 64),
    # pairs, tiles without a partner, single tiles >= 16 and rows of two and three chunks
    "mixed_long": lambda: synth.custom_workload([1] * 12, [99, 2500, 300, 4300, 128, 129, 2047, 2048, 2049, 5000, 1, 640], 4, 2, 128, 64),
    "d64_mixed": lambda: synth.custom_workload([1] * 20, _lens(2, 20, 1, 3000), 6, 3, 64, 32),
    "g1_single_head": lambda: synth.custom_workload([1] * 7, [4500, 130, 2300, 64, 1000, 3000, 257], 2, 2, 128, 16),
    "one_sequence": lambda: synth.custom_workload([1], [3333], 16, 2, 128, 64),
}


@pytest.mark.parametrize("name", list(CASES))
def test_train_fwd_persistent_equals_per_item_schedule(tik, name):
    w = CASES[name]()
    q, k, v, cu = synth.make_qkv(w, "cuda")
    mx = max(w.seq_lens)
    lse_a = torch.full((w.total_tokens, w.Hq), -1.0, dtype=torch.float32, device="cuda")
    lse_b = torch.full_like(lse_a, -2.0)
    o_a = tik.tik_attn_train_fwd(q, k, v, cu, mx, w.softmax_scale, o=torch.full_like(q, 7.0), lse=lse_a)
    o_b = tik.tik_attn_train_fwd(q, k, v, cu, mx, w.softmax_scale, o=torch.full_like(q, 9.0), lse=lse_b, ws=False)
    assert count_diff(o_a, o_b) == 0
    assert count_diff(lse_a, lse_b) == 0
    # an inflated length bound (more candidate items per sequence, all empty) changes nothing
    o_c = tik.tik_attn_train_fwd(q, k, v, cu, mx + 5000, w.softmax_scale)
    assert count_diff(o_a, o_c) == 0
    if w.total_tokens <= 20000:
        ref, _ = oracle.attn_packed(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(),
                                    w.cu_seqlens(), w.softmax_scale)
        assert np.abs(o_a.float().cpu().numpy() - ref).max() <= ATTN_TOL


def test_empty_sequences_in_the_pack(tik):
    """Zero-length entries of cu_seqlens produce no work item and leave every other row alone."""
    w = synth.custom_workload([1, 1, 1], [299, 40, 2100], 8, 1, 128, 64)
    q, k, v, _ = synth.make_qkv(w, "cuda")
    L = w.seq_lens
    cu = torch.tensor([0, 0, L[0], L[0], L[0] + L[1], L[0] + L[1], sum(L), sum(L)], dtype=torch.int32, device="cuda")
    o_a = tik.tik_attn_train_fwd(q, k, v, cu, max(L), w.softmax_scale)
    o_b = tik.tik_attn_train_fwd(q, k, v, cu, max(L), w.softmax_scale, ws=False)
    o_c = tik.tik_attn_train_fwd(q, k, v, torch.from_numpy(w.cu_seqlens()).cuda(), max(L), w.softmax_scale)
    assert count_diff(o_a, o_b) == 0 and count_diff(o_a, o_c) == 0


@pytest.mark.parametrize("page", [16, 64, 128])
def test_prefill_persistent_equals_per_item_schedule(tik, page):
    """Whole prompts and prompts behind cached prefixes of odd lengths, several per CTA."""
    P = [700, 130, 2500, 64, 1, 1025, 4200, 333, 128, 2048, 90, 1500]
    w = synth.custom_workload(P, [1] * len(P), 8, 2, 128, page)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros(layout.num_pages, w.Hkv, page, w.d, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    tik.tik_kv_cache_write(k, v, cu, torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda"), kc, vc, bt)
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale)
    cu_h = w.cu_seqlens()
    for start in ([0] * len(P), [p // 3 for p in P], [min(p - 1, 129) for p in P]):
        rows = torch.cat([torch.arange(cu_h[s] + a, cu_h[s] + p) for s, (a, p) in enumerate(zip(start, P))]).cuda()
        lens = [p - a for a, p in zip(start, P)]
        cu_q = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
        ctx = torch.tensor(P, dtype=torch.int32, device="cuda")
        qn = q[rows].contiguous()
        o_a = tik.tik_attn_prefill(qn, cu_q, ctx, kc, vc, bt, max(lens), max(P), w.softmax_scale)
        o_b = tik.tik_attn_prefill(qn, cu_q, ctx, kc, vc, bt, max(lens), max(P), w.softmax_scale, ws=False)
        assert count_diff(o_a, o_b) == 0
        assert count_diff(o_a, o_train[rows]) == 0


def test_caller_scratch_is_used_and_too_small_scratch_falls_back(tik):
    w = synth.custom_workload([1] * 5, [300, 900, 20, 2600, 77], 8, 2, 128, 64)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    mx = max(w.seq_lens)
    need = tik.workspace_bytes(tik.OP_ATTN_TRAIN_FWD, w.S, max_ctx=mx)
    assert need > 16
    ws = torch.zeros(need + 64, dtype=torch.uint8, device="cuda")
    ws[need:] = 0x5A
    o_a = tik.tik_attn_train_fwd(q, k, v, cu, mx, w.softmax_scale, ws=ws)
    assert int(ws[:4].view(torch.int32).item()) > 0          # the plan's entry count was written
    assert bool((ws[need:] == 0x5A).all())
    small = torch.zeros(32, dtype=torch.uint8, device="cuda")
    o_b = tik.tik_attn_train_fwd(q, k, v, cu, mx, w.softmax_scale, ws=small)
    assert bool((small == 0).all())                          # not touched: the per-item schedule ran
    assert count_diff(o_a, o_b) == 0
    # a call with fewer work items than two per SM also runs per item, whatever scratch it is given
    w1 = synth.custom_workload([1], [700], 4, 2, 128, 64)
    q1, k1, v1, cu1 = synth.make_qkv(w1, "cuda")
    ws1 = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    o1 = tik.tik_attn_train_fwd(q1, k1, v1, cu1, 701, w1.softmax_scale, ws=ws1)
    assert bool((ws1 == 0).all())
    assert count_diff(o1, tik.tik_attn_train_fwd(q1, k1, v1, cu1, 701, w1.softmax_scale, ws=False)) == 0
