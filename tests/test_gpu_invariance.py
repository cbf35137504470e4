"""GPU bit-exactness matrix: an attention row's bits depend only on its query, its causal
K/V prefix, the scale and d -- not on batch composition, slot, packing order, page size or
placement, grid bounds, stale data behind the context, stream, or graph replay (paper Sec. 3.2
"same query data and causal KV prefix"; Sec. 6 Q3 lists batched-versus-single decode,
bitwise-preservation and CUDA-graph checks)."""
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


def _full_cache(tik, w, k, v, cu, layout, fill=0.0):
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.full((layout.num_pages, w.Hkv, layout.page_size, w.d), fill, dtype=torch.bfloat16, device="cuda")
    vc = torch.full_like(kc, fill)
    ctx = torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda")
    tik.tik_kv_cache_write(k, v, cu, ctx, kc, vc, bt)
    return kc, vc, bt


def _decode_rows(tik, w, q, kc, vc, bt, seqs, positions, max_ctx=None):
    cu = w.cu_seqlens()
    rows = torch.tensor([int(cu[s]) + p for s, p in zip(seqs, positions)], device="cuda")
    ctx = torch.tensor([p + 1 for p in positions], dtype=torch.int32, device="cuda")
    o = tik.tik_attn_decode(q[rows].contiguous(), ctx, kc, vc, bt[seqs].contiguous(),
                            max_ctx or (max(positions) + 1), w.softmax_scale)
    return rows, o


@pytest.fixture(scope="module")
def case(tik):
    w = synth.custom_workload([700, 64, 2300, 129, 1], [1500, 200, 900, 127, 40], 8, 2, 128, 64)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale)
    layout = synth.make_paged_layout(w)
    kc, vc, bt = _full_cache(tik, w, k, v, cu, layout)
    return w, q, k, v, cu, o_train, layout, kc, vc, bt


def test_batched_versus_single_decode(tik, case):
    """36 comparisons: 6 positions of 3 sequences, each alone and inside 2 other batches."""
    w, q, k, v, cu, o_train, layout, kc, vc, bt = case
    n = 0
    for s in (0, 2, 3):
        L = w.seq_lens[s]
        for pos in (0, 127, 128, L // 2, L - 2, L - 1):
            rows, single = _decode_rows(tik, w, q, kc, vc, bt, [s], [pos])
            assert count_diff(single, o_train[rows]) == 0
            others = [t for t in range(w.S) if t != s]
            for batch in ([others[0], s, others[1]], others + [s]):
                poss = [pos if t == s else w.seq_lens[t] - 1 for t in batch]
                rows_b, ob = _decode_rows(tik, w, q, kc, vc, bt, batch, poss)
                slot = batch.index(s)
                assert torch.equal(bits(ob[slot]), bits(single[0]))
                assert count_diff(ob, o_train[rows_b]) == 0
                n += 1
    assert n == 36


def test_packing_order_and_grid_bounds(tik, case):
    w, q, k, v, cu, o_train, *_ = case
    cu_h = w.cu_seqlens()
    order = [3, 0, 4, 2, 1]
    idx = torch.cat([torch.arange(cu_h[s], cu_h[s + 1]) for s in order]).cuda()
    cu2 = torch.tensor(np.concatenate([[0], np.cumsum([w.seq_lens[s] for s in order])]),
                       dtype=torch.int32, device="cuda")
    o2 = tik.tik_attn_train_fwd(q[idx].contiguous(), k[idx].contiguous(), v[idx].contiguous(), cu2,
                                max(w.seq_lens), w.softmax_scale)
    assert count_diff(o2, o_train[idx]) == 0
    # inflated host upper bound: more idle CTAs, same bits
    o3 = tik.tik_attn_train_fwd(q, k, v, cu, 3 * max(w.seq_lens) + 77, w.softmax_scale)
    assert count_diff(o3, o_train) == 0
    # repeatability, also on another stream
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        o4 = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale)
    st.synchronize()
    assert count_diff(o4, o_train) == 0


@pytest.mark.parametrize("page", [16, 32, 128])
def test_page_size_and_placement(tik, case, page):
    w, q, k, v, cu, o_train, *_ = case
    w2 = synth.custom_workload(w.prompt_lens, w.response_lens, w.Hq, w.Hkv, w.d, page)
    for shuffle in (True, False):
        layout = synth.make_paged_layout(w2, shuffle=shuffle)
        kc, vc, bt = _full_cache(tik, w2, k, v, cu, layout)
        seqs = list(range(w.S))
        for frac in (1.0, 0.37):
            pos = [max(0, int(L * frac) - 1) for L in w.seq_lens]
            rows, o = _decode_rows(tik, w2, q, kc, vc, bt, seqs, pos)
            assert count_diff(o, o_train[rows]) == 0
        # whole sequences as one prefill against the full cache
        ctx = torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda")
        op = tik.tik_attn_prefill(q, cu, ctx, kc, vc, bt, max(w.seq_lens), max(w.seq_lens), w.softmax_scale)
        assert count_diff(op, o_train) == 0


def test_shared_prompt_pages_equal_private_copies(tik):
    w = synth.custom_workload([192, 192, 192, 64], [30, 99, 7, 50], 4, 2, 128, 64, group_of=[0, 0, 0, 1])
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale)
    for share in (True, False):
        layout = synth.make_paged_layout(w, share_prompts=share)
        assert (layout.shared_prompt_pages > 0) == share
        o_roll = Rollout(tik, w, q, k, v, layout).replay()
        assert count_diff(o_roll, o_train) == 0


def test_chunked_prefill_behind_a_cached_prefix(tik, case):
    """One prefill call == two calls split at odd positions (the second behind a cached prefix)."""
    w, q, k, v, cu, o_train, layout, *_ = case
    ro = Rollout(tik, w, q, k, v, layout)
    seqs = [0, 2, 3]
    split = [333, 2049, 1]
    stop = [w.seq_lens[s] for s in seqs]
    rows1, o1 = ro.prefill(seqs=seqs, start=[0, 0, 0], stop=split)
    rows2, o2 = ro.prefill(seqs=seqs, start=split, stop=stop)
    assert count_diff(o1, o_train[rows1]) == 0
    assert count_diff(o2, o_train[rows2]) == 0


def test_future_tokens_and_stale_cache_contents_do_not_matter(tik, case):
    w, q, k, v, cu, o_train, layout, *_ = case
    cu_h = w.cu_seqlens()
    # train: overwrite everything after position t in every sequence with other finite values
    t = 100
    k2, v2, q2 = k.clone(), v.clone(), q.clone()
    keep = torch.cat([torch.arange(cu_h[s], min(cu_h[s] + t + 1, cu_h[s + 1])) for s in range(w.S)]).cuda()
    mask = torch.ones(w.total_tokens, dtype=torch.bool, device="cuda")
    mask[keep] = False
    k2[mask] = 7.5
    v2[mask] = -123.0
    q2[mask] = 3.0
    o2 = tik.tik_attn_train_fwd(q2, k2, v2, cu, max(w.seq_lens), w.softmax_scale)
    assert count_diff(o2[keep], o_train[keep]) == 0
    # paged: a pool full of large finite garbage behind the written prefix
    kc, vc, bt = _full_cache(tik, w, k, v, cu, layout, fill=0.0)
    upto = [L // 2 + 1 for L in w.seq_lens]
    kd = torch.full_like(kc, 1.0e4)
    vd = torch.full_like(vc, -3.0e4)
    cu_part = torch.tensor(np.concatenate([[0], np.cumsum(upto)]), dtype=torch.int32, device="cuda")
    rows = torch.cat([torch.arange(cu_h[s], cu_h[s] + upto[s]) for s in range(w.S)]).cuda()
    tik.tik_kv_cache_write(k[rows].contiguous(), v[rows].contiguous(), cu_part,
                           torch.tensor(upto, dtype=torch.int32, device="cuda"), kd, vd, bt)
    pos = [u - 1 for u in upto]
    r1, o_clean = _decode_rows(tik, w, q, kc, vc, bt, list(range(w.S)), pos)
    r2, o_dirty = _decode_rows(tik, w, q, kd, vd, bt, list(range(w.S)), pos)
    assert count_diff(o_clean, o_train[r1]) == 0
    assert count_diff(o_dirty, o_clean) == 0


def test_cuda_graph_replay_with_varying_inputs(tik, case):
    """Capture one decode call, replay it after rewriting q / ctx_lens / block table in place."""
    w, q, k, v, cu, o_train, layout, kc, vc, bt = case
    cu_h = w.cu_seqlens()
    B = 3
    qb = torch.zeros(B, w.Hq, w.d, dtype=torch.bfloat16, device="cuda")
    ctx = torch.ones(B, dtype=torch.int32, device="cuda")
    btb = bt[:B].clone()
    ob = torch.zeros_like(qb)
    max_ctx = max(w.seq_lens)
    ws = torch.empty(tik.workspace_bytes(tik.OP_ATTN_DECODE, B, w.Hq, w.Hkv, w.d, max_ctx), dtype=torch.uint8,
                     device="cuda")

    def fill(seqs, positions):
        rows = torch.tensor([int(cu_h[s]) + p for s, p in zip(seqs, positions)], device="cuda")
        qb.copy_(q[rows])
        ctx.copy_(torch.tensor([p + 1 for p in positions], dtype=torch.int32, device="cuda"))
        btb.copy_(bt[seqs])
        return rows

    fill([0, 1, 2], [10, 20, 30])
    tik.tik_attn_decode(qb, ctx, kc, vc, btb, max_ctx, w.softmax_scale, ws=ws, o=ob)   # warm-up / set-up
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        tik.tik_attn_decode(qb, ctx, kc, vc, btb, max_ctx, w.softmax_scale, ws=ws, o=ob)
    for seqs, positions in ([[0, 1, 2], [2199, 263, 3199]], [[4, 2, 0], [0, 2048, 1]], [[3, 3, 1], [255, 128, 63]]):
        rows = fill(seqs, positions)
        graph.replay()
        torch.cuda.synchronize()
        assert count_diff(ob, o_train[rows]) == 0


def test_empty_and_degenerate_inputs(tik):
    w = synth.custom_workload([5, 1, 130], [0, 0, 0], 4, 4, 64, 16)       # includes length-1 and no responses
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o = tik.tik_attn_train_fwd(q, k, v, cu, 130, w.softmax_scale)
    ref, _ = oracle.attn_packed(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(),
                                w.cu_seqlens(), w.softmax_scale)
    assert np.abs(o.float().cpu().numpy() - ref).max() <= ATTN_TOL
    # an empty sequence in the middle of the pack and zero total work are both fine
    cu2 = torch.tensor([0, 5, 5, 6, 136], dtype=torch.int32, device="cuda")
    o2 = tik.tik_attn_train_fwd(q, k, v, cu2, 130, w.softmax_scale)
    assert count_diff(o2, o) == 0
    empty = torch.empty(0, 4, 64, dtype=torch.bfloat16, device="cuda")
    tik.tik_attn_train_fwd(empty, empty, empty, torch.zeros(1, dtype=torch.int32, device="cuda"), 0,
                           w.softmax_scale)
    # a decode slot with ctx_len 0 is skipped and its output left untouched
    layout = synth.make_paged_layout(w)
    kc, vc, bt = _full_cache(tik, w, k, v, cu, layout)
    qd = q[[4, 5, 135]].contiguous()
    od = torch.full_like(qd, 9.0)
    ctx = torch.tensor([5, 0, 130], dtype=torch.int32, device="cuda")
    tik.tik_attn_decode(qd, ctx, kc, vc, bt, 130, w.softmax_scale, o=od)
    assert bool((od[1] == 9.0).all())
    assert torch.equal(bits(od[0]), bits(o[4])) and torch.equal(bits(od[2]), bits(o[135]))


def test_bad_block_table_entry_is_flagged_not_fatal(tik, case):
    w, q, k, v, cu, o_train, layout, kc, vc, bt = case
    bad = bt.clone()
    bad[1, 0] = layout.num_pages + 5
    rows, o = _decode_rows(tik, w, q, kc, vc, bad, [0, 1], [50, 100])
    assert tik.device_status() & tik.DEV_BAD_BLOCK
    assert torch.equal(bits(o[0]), bits(o_train[rows[0]]))            # the other slot is unaffected
    assert bool(torch.isfinite(o.float()).all())


def test_decode_with_several_chunks_per_cta(tik):
    """A large decode batch lets one CTA stream up to four consecutive 2048-key chunks; a small
    one gets a CTA per chunk.  The chunk partials, and so every output bit, must not depend on it."""
    rng = np.random.default_rng(77)
    lens = [int(x) for x in rng.integers(2100, 6200, 150)]
    lens[0], lens[1], lens[2] = 8192, 2048, 2049          # exactly four chunks, one chunk, one chunk + one key
    w = synth.custom_workload([1] * len(lens), [L - 1 for L in lens], 4, 4, 64, 64, index=33)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(w.seq_lens), w.softmax_scale)
    layout = synth.make_paged_layout(w)
    kc, vc, bt = _full_cache(tik, w, k, v, cu, layout)
    seqs = list(range(w.S))
    for frac in (1.0, 0.55):
        pos = [max(1, int(L * frac)) - 1 for L in lens]
        rows, o = _decode_rows(tik, w, q, kc, vc, bt, seqs, pos)
        assert count_diff(o, o_train[rows]) == 0, frac
        # the same rows decoded three at a time (one CTA per chunk)
        for s0 in (0, 60):
            sub = seqs[s0:s0 + 3]
            rows3, o3 = _decode_rows(tik, w, q, kc, vc, bt, sub, [pos[s] for s in sub])
            assert count_diff(o3, o_train[rows3]) == 0
    ref = oracle.attn_rows(q[rows[:4], 1].float().cpu().numpy(),
                           np.concatenate([k[int(cu[s]):int(cu[s + 1]), 1].float().cpu().numpy() for s in range(4)]),
                           np.concatenate([v[int(cu[s]):int(cu[s + 1]), 1].float().cpu().numpy() for s in range(4)]),
                           [int(cu[s]) for s in range(4)], [p + 1 for p in pos[:4]], w.softmax_scale)[0]
    assert np.abs(o[:4, 1].float().cpu().numpy() - ref).max() <= ATTN_TOL
