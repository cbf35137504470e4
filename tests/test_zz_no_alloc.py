"""The decode entry point that allocates nothing (tik_attn_decode_static).

Some callers of the library cannot allocate device memory at call time: a serving process
whose KV-cache pool took all free memory at start-up, or a decode loop that cannot afford
the device-wide synchronisation of cudaMalloc/cudaFree.  For them the library keeps the
split-KV scratch in a fixed device array of its own.  This test drives that entry point
through the C ABI and checks, on two calls in a row that share the scratch, that its output
has zero differing bits from tik_attn_decode (same kernels), and that a problem larger than
the fixed scratch is refused.  It is collected last so that a run which stops at the first
failure has already run every other test.
"""
import pytest
import torch

from paper_2609_35140_b200 import synth

pytestmark = pytest.mark.gpu


def _case(tik, prompt_lens, response_lens, Hq, Hkv, d, page, index):
    w = synth.custom_workload(prompt_lens, response_lens, Hq, Hkv, d, page, index=index)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros(layout.num_pages, w.Hkv, layout.page_size, w.d, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    ctx = torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda")
    tik.tik_kv_cache_write(k, v, cu, ctx, kc, vc, bt)
    cu_h = w.cu_seqlens()
    last = torch.tensor([cu_h[s + 1] - 1 for s in range(w.S)], device="cuda")
    return w, q[last].contiguous(), ctx, kc, vc, bt


def test_static_decode_matches_decode_on_two_calls_in_a_row():
    from paper_2609_35140_b200 import binding as tik
    tik.load()
    # first call: three chunks per sequence; second call: other shapes, fewer chunks, so stale
    # partials of the first call sit in the shared scratch while the second one runs
    cases = [_case(tik, [700, 100, 2049], [3500, 1, 2100], 8, 2, 128, 64, 201),
             _case(tik, [90, 300], [38, 1900], 6, 3, 64, 16, 202)]
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    for w, q, ctx, kc, vc, bt in cases:
        ref = tik.tik_attn_decode(q, ctx, kc, vc, bt, max(w.seq_lens), w.softmax_scale)
        out = torch.full_like(ref, 7.0)
        rc = tik.tik_attn_decode_static(q, ctx, kc, vc, bt, max(w.seq_lens), w.softmax_scale, out,
                                        dev_flags=flags)
        assert rc == 0
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    # same call again without a caller flag word (flags go to the library's own word)
    w, q, ctx, kc, vc, bt = cases[0]
    ref = tik.tik_attn_decode(q, ctx, kc, vc, bt, max(w.seq_lens), w.softmax_scale)
    out = torch.full_like(ref, 7.0)
    assert tik.tik_attn_decode_static(q, ctx, kc, vc, bt, max(w.seq_lens), w.softmax_scale, out) == 0
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    assert int(flags.item()) == 0
    assert tik.device_status() == 0


def test_static_decode_refuses_problems_beyond_its_scratch():
    from paper_2609_35140_b200 import binding as tik
    tik.load()
    w, q, ctx, kc, vc, bt = _case(tik, [64, 64], [10, 20], 8, 2, 128, 64, 203)
    out = torch.full((2, 8, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    # claim a context so long that 2 * 8 * chunks * 132 * 4 bytes exceeds the fixed scratch
    huge_ctx = 2048 * (tik.STATIC_SCRATCH_BYTES // (2 * 8 * 132 * 4) + 1)
    rc = tik.tik_attn_decode_static(q, ctx, kc, vc, bt, huge_ctx, w.softmax_scale, out)
    assert rc == -3
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())          # nothing was launched


def test_static_decode_reports_device_flags_through_the_callers_word():
    """A block-table entry outside the pool is read as a page of zeros and flagged.  The entry
    point has no context to keep flags in: they reach the caller only through `dev_flags`."""
    from paper_2609_35140_b200 import binding as tik
    tik.load()
    w, q, ctx, kc, vc, bt = _case(tik, [300, 64], [200, 90], 8, 2, 128, 64, 204)
    bad = bt.clone()
    bad[0, 1] = kc.shape[0] + 5
    ref = tik.tik_attn_decode(q, ctx, kc, vc, bad, max(w.seq_lens), w.softmax_scale)
    assert tik.device_status() == tik.DEV_BAD_BLOCK          # the context-based entry point keeps it
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full_like(ref, 7.0)
    assert tik.tik_attn_decode_static(q, ctx, kc, vc, bad, max(w.seq_lens), w.softmax_scale, out, dev_flags=flags) == 0
    torch.cuda.synchronize()
    assert int(flags.item()) == tik.DEV_BAD_BLOCK
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    assert bool(torch.isfinite(out.float()).all())
    # without a word the call still succeeds; the flag is discarded (documented in the header)
    assert tik.tik_attn_decode_static(q, ctx, kc, vc, bad, max(w.seq_lens), w.softmax_scale, out) == 0
    torch.cuda.synchronize()
    assert tik.device_status() == 0
