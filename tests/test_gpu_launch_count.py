"""The library's own kernel-launch counter (what `bench.py` reports as `gpu_launches`): every entry
point adds exactly the kernels it enqueues -- one for a decode whose contexts fit one 2048-key chunk
(it normalises and stores its rows itself), two when a combine follows; one for a small packed
forward, two or more when the persistent schedule (work-list kernel + attention kernel) runs; two
for the token log-prob (GEMM + finish) -- and the one-chunk decode gives the bits of the same rows
computed with a larger host bound (partials + combine)."""
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


def _delta(tik, fn):
    n0 = tik.kernel_launches()
    out = fn()
    return tik.kernel_launches() - n0, out


def test_every_entry_point_counts_its_kernels(tik):
    Hq, Hkv, d, page = 8, 2, 128, 64
    lens = [700, 1500, 2048, 90]
    w = synth.custom_workload([1] * len(lens), [L - 1 for L in lens], Hq, Hkv, d, page)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    n_train, o_train = _delta(tik, lambda: tik.tik_attn_train_fwd(q, k, v, cu, max(lens), w.softmax_scale, ws=False))
    assert n_train == 1                                        # no scratch: one CTA per work item
    n_plan, o_plan = _delta(tik, lambda: tik.tik_attn_train_fwd(q, k, v, cu, max(lens), w.softmax_scale))
    assert n_plan in (1, 2) and count_diff(o_plan, o_train) == 0   # with scratch: work list + persistent kernel, or the same kernel
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros((layout.num_pages, Hkv, page, d), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    ctx = torch.tensor(lens, dtype=torch.int32, device="cuda")
    n_kv, _ = _delta(tik, lambda: tik.tik_kv_cache_write(k, v, cu, ctx, kc, vc, bt))
    assert n_kv == 1
    cu_h = w.cu_seqlens()
    rows = torch.tensor([int(cu_h[s]) + L - 1 for s, L in enumerate(lens)], device="cuda")
    qd = q[rows].contiguous()
    # contexts of at most one chunk: the decode kernel alone
    n_one, o_one = _delta(tik, lambda: tik.tik_attn_decode(qd, ctx, kc, vc, bt, 2048, w.softmax_scale))
    assert n_one == 1
    assert count_diff(o_one, o_train[rows]) == 0
    # the same contexts under a host bound of two chunks: partials and the combine kernel, same bits
    bt2 = torch.cat([bt, torch.full((len(lens), 2048 // page), -1, dtype=torch.int32, device="cuda")], dim=1).contiguous()
    n_two, o_two = _delta(tik, lambda: tik.tik_attn_decode(qd, ctx, kc, vc, bt2, 4096, w.softmax_scale))
    assert n_two == 2
    assert count_diff(o_two, o_one) == 0
    # token log-prob: the fused GEMM and the finish kernel
    g = torch.Generator(device="cuda").manual_seed(5)
    x = (torch.randn(40, 256, generator=g, device="cuda")).to(torch.bfloat16)
    W = (torch.randn(2048, 256, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    tgt = torch.randint(0, 2048, (40,), generator=g, device="cuda").to(torch.int32)
    n_lp, _ = _delta(tik, lambda: tik.tik_token_logprob(x, W, tgt))
    assert n_lp == 2
    n_lin, _ = _delta(tik, lambda: tik.tik_linear(x, W))
    assert n_lin == 1
    assert isinstance(tik.kernel_launches(), int) and tik.kernel_launches() >= n_train + n_plan + n_kv + n_one + n_two + n_lp + n_lin
