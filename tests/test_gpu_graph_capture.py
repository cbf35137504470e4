"""The rollout-side entry points can be captured into a CUDA graph (nothing in a call allocates,
synchronises or reads the device from the host): a graph of cache write + decode, replayed after
the inputs were changed in place, gives the bits of the eager calls on the new inputs -- contexts
of one chunk (the decode kernel finishes its rows itself) and of several (partials + combine)."""
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


@pytest.mark.parametrize("lens", [[300, 1024, 2047, 65], [2500, 4096, 900, 5000]])
def test_cache_write_and_decode_replay_from_a_graph(tik, lens):
    Hq, Hkv, d, page = 16, 4, 128, 64
    S = len(lens)
    # every sequence holds one token more than its context: the graph writes that token and decodes it
    w = synth.custom_workload([1] * S, [L for L in lens], Hq, Hkv, d, page)
    q, k, v, cu = synth.make_qkv(w, "cuda")
    layout = synth.make_paged_layout(w)
    bt = torch.from_numpy(layout.block_table).cuda()
    kc = torch.zeros((layout.num_pages, Hkv, page, d), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    cu_h = w.cu_seqlens()
    full = torch.tensor([L + 1 for L in lens], dtype=torch.int32, device="cuda")
    tik.tik_kv_cache_write(k, v, cu, full, kc, vc, bt)                 # all L + 1 tokens once, eagerly
    o_ref = tik.tik_attn_train_fwd(q, k, v, cu, max(lens) + 1, w.softmax_scale)

    # static buffers of the graph: the step's token rows, its context lengths, its output
    step_rows = torch.tensor([int(cu_h[s]) + lens[s] - 1 for s in range(S)], device="cuda")     # second-to-last token
    qs, ks, vs = q[step_rows].clone(), k[step_rows].clone(), v[step_rows].clone()
    ctx = torch.tensor(lens, dtype=torch.int32, device="cuda")
    cu1 = torch.arange(S + 1, dtype=torch.int32, device="cuda")
    o = torch.empty(S, Hq, d, dtype=torch.bfloat16, device="cuda")
    max_ctx = max(lens) + 1
    ws = torch.empty(tik.workspace_bytes(tik.OP_ATTN_DECODE, S, Hq, Hkv, d, max_ctx), dtype=torch.uint8, device="cuda")

    def step():
        tik.tik_kv_cache_write(ks, vs, cu1, ctx, kc, vc, bt)
        tik.tik_attn_decode(qs, ctx, kc, vc, bt, max_ctx, w.softmax_scale, ws=ws, o=o)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                                         # once eagerly: launch set-up is done
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    assert count_diff(o, o_ref[step_rows]) == 0
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    # replay on the NEXT token: new rows and context lengths written into the graph's buffers
    next_rows = step_rows + 1
    qs.copy_(q[next_rows]); ks.copy_(k[next_rows]); vs.copy_(v[next_rows])
    ctx.add_(1)
    o.fill_(7.0)
    g.replay()
    torch.cuda.synchronize()
    assert count_diff(o, o_ref[next_rows]) == 0
    assert tik.device_status() == 0
