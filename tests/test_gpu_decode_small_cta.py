"""Decode through the small-CTA kernel (two CTAs per SM, 8-row query atoms read through a
zero-stride descriptor, weights written over the scores).  The library picks it when a call has
at most one (sequence, KV head) pair per SM and about as many 2048-key chunks as SMs or more;
the shapes below are in that range (80-120 pairs, two or three chunks each).  Its rows must equal
the packed train-forward's rows bit for bit, for every group size it serves, both head sizes and
several page sizes, with ragged contexts, batch slots without work and a stale cache."""
import numpy as np
import pytest
import torch

from paper_2609_35140_b200 import synth
from gpu_common import count_diff

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tik():
    from paper_2609_35140_b200 import binding
    binding.load()
    yield binding
    assert binding.device_status() == 0


def _lens(seed, n, lo, hi):
    return [int(x) for x in np.random.default_rng(seed).integers(lo, hi + 1, n)]


@pytest.mark.parametrize("G,Hkv,d,page,S", [(1, 4, 128, 64, 24), (4, 4, 128, 16, 20), (7, 4, 128, 64, 20),
                                            (8, 5, 128, 128, 24), (3, 4, 64, 32, 30), (8, 2, 64, 64, 40)])
def test_small_cta_decode_equals_train_rows(tik, G, Hkv, d, page, S):
    lens = _lens(100 + G + d, S, 2049, 4700)
    lens[0], lens[1], lens[2] = 2049, 4096, 4097            # chunk boundaries
    w = synth.custom_workload([1] * S, [L - 1 for L in lens], G * Hkv, Hkv, d, page)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(lens), w.softmax_scale)
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.full((layout.num_pages, Hkv, page, d), 2.0, dtype=torch.bfloat16, device="cuda")   # stale finite values
    vc = torch.full_like(kc, -3.0)
    tik.tik_kv_cache_write(k, v, cu, torch.tensor(lens, dtype=torch.int32, device="cuda"), kc, vc, bt)
    cu_h = w.cu_seqlens()
    for frac in (1.0, 0.71):
        pos = [max(2049, int(L * frac)) - 1 for L in lens]
        ctx = [p + 1 for p in pos]
        ctx[3] = 0                                           # a batch slot without work: its output row stays
        rows = torch.tensor([int(cu_h[s]) + p for s, p in enumerate(pos)], device="cuda")
        o = torch.full((S, w.Hq, d), 7.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(S, w.Hq, dtype=torch.float32, device="cuda")
        tik.tik_attn_decode(q[rows].contiguous(), torch.tensor(ctx, dtype=torch.int32, device="cuda"), kc, vc, bt,
                            max(ctx), w.softmax_scale, o=o, lse=lse)
        keep = [s for s in range(S) if s != 3]
        assert count_diff(o[keep], o_train[rows][keep]) == 0, frac
        assert bool((o[3] == 7.0).all())
        assert bool(torch.isfinite(lse[keep]).all())
    # one sequence alone (few chunks: the one-CTA-per-SM kernel) gives the same bits as inside the batch
    s = 2
    o1 = tik.tik_attn_decode(q[int(cu_h[s]) + lens[s] - 1][None].contiguous(),
                             torch.tensor([lens[s]], dtype=torch.int32, device="cuda"), kc, vc, bt[s][None].contiguous(),
                             lens[s], w.softmax_scale)
    assert count_diff(o1[0], o_train[int(cu_h[s]) + lens[s] - 1]) == 0


@pytest.mark.parametrize("S,Hkv,G,lo,hi", [(150, 8, 2, 2049, 4096),     # 1200 pairs x 2 chunks: one CTA walks both chunks
                                           (160, 4, 4, 1, 2048),        # 640 pairs x 1 chunk: the kernel finishes its rows itself
                                           (40, 8, 1, 2049, 4000)])     # 320 pairs x 2 chunks, one chunk per CTA
def test_small_cta_decode_with_more_pairs_than_sms(tik, S, Hkv, G, lo, hi):
    """Contexts of at most two chunks take the small-CTA kernel whatever the number of (sequence,
    KV head) pairs; the rows equal the packed train-forward's rows bit for bit."""
    d, page = 128, 64
    lens = _lens(7 * S + G, S, lo, hi)
    lens[0], lens[1] = lo, hi
    w = synth.custom_workload([1] * S, [L - 1 for L in lens], G * Hkv, Hkv, d, page)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    o_train = tik.tik_attn_train_fwd(q, k, v, cu, max(lens), w.softmax_scale)
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros((layout.num_pages, Hkv, page, d), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    ctx = torch.tensor(lens, dtype=torch.int32, device="cuda")
    tik.tik_kv_cache_write(k, v, cu, ctx, kc, vc, bt)
    cu_h = w.cu_seqlens()
    rows = torch.tensor([int(cu_h[s]) + lens[s] - 1 for s in range(S)], device="cuda")
    lse = torch.zeros(S, w.Hq, dtype=torch.float32, device="cuda")
    lse_train = torch.zeros(q.shape[0], w.Hq, dtype=torch.float32, device="cuda")
    tik.tik_attn_train_fwd(q, k, v, cu, max(lens), w.softmax_scale, lse=lse_train)
    n0 = tik.kernel_launches()
    o = tik.tik_attn_decode(q[rows].contiguous(), ctx, kc, vc, bt, max(lens), w.softmax_scale, lse=lse)
    assert tik.kernel_launches() - n0 == (1 if max(lens) <= 2048 else 2)
    assert count_diff(o, o_train[rows]) == 0
    assert count_diff(lse, lse_train[rows]) == 0
