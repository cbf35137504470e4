"""The seeded workload generators: shapes, length mixes and page layouts."""
import numpy as np
import torch

from paper_2609_35140_b200 import synth


def test_workload_shapes_follow_the_benchmark_configs():
    w = [synth.get_workload(i) for i in range(5)]
    assert (w[0].Hq, w[0].Hkv, w[0].d, w[0].page_size) == (4, 1, 64, 16)
    assert w[0].seq_lens == [96, 160] and (w[0].hidden, w[0].vocab) == (256, 2048)
    assert (w[1].Hq, w[1].Hkv, w[1].S) == (12, 2, 16) and all(128 <= r <= 2048 for r in w[1].response_lens)
    assert w[2].S == 64 and w[2].group_of[7] == 0 and w[2].group_of[8] == 1
    assert all(256 <= r <= 4096 for r in w[2].response_lens) and w[2].vocab == 152064
    assert w[3].seq_lens == [16384] * 16 and w[3].decode_contexts == [4096, 8192, 16384]
    assert w[4].S == 256 and max(w[4].response_lens) <= 8192 and min(w[4].response_lens) >= 16
    assert 1200 < np.mean(w[4].response_lens) < 2800
    # seeded: the same draw every time
    assert synth.get_workload(1).response_lens == w[1].response_lens


def test_group_members_share_their_prompt():
    w = synth.custom_workload([40, 40, 24], [5, 9, 3], 4, 2, 64, 16, group_of=[0, 0, 1])
    q, k, v, cu = synth.make_qkv(w)
    cu = cu.numpy()
    assert torch.equal(k[cu[0]:cu[0] + 40], k[cu[1]:cu[1] + 40])
    assert not torch.equal(k[cu[0] + 40:cu[0] + 45], k[cu[1] + 40:cu[1] + 45])
    layout = synth.make_paged_layout(w)
    assert (layout.block_table[0, :2] == layout.block_table[1, :2]).all()      # 2 whole prompt pages
    assert layout.block_table[0, 2] != layout.block_table[1, 2]
    assert layout.shared_prompt_pages == 2


def test_paged_layout_is_a_valid_placement():
    for i in (0, 1, 2):
        w = synth.get_workload(i)
        layout = synth.make_paged_layout(w)
        used = layout.block_table[layout.block_table >= 0]
        assert used.max() < layout.num_pages
        owners = {}
        for s in range(w.S):
            n = -(-w.seq_lens[s] // layout.page_size)
            assert (layout.block_table[s, :n] >= 0).all() and (layout.block_table[s, n:] == -1).all()
            for b in range(n):
                owners.setdefault(int(layout.block_table[s, b]), set()).add(w.group_of[s])
        assert all(len(g) == 1 for g in owners.values())     # pages never cross groups


def test_fill_paged_cache_round_trips():
    w = synth.get_workload(0)
    q, k, v, cu = synth.make_qkv(w)
    layout = synth.make_paged_layout(w)
    kc, vc = synth.fill_paged_cache(w, layout, k, v)
    cu = cu.numpy()
    for s in range(w.S):
        for t in (0, 15, 16, w.seq_lens[s] - 1):
            page = layout.block_table[s, t // 16]
            assert torch.equal(kc[page, :, t % 16], k[cu[s] + t])
            assert torch.equal(vc[page, :, t % 16], v[cu[s] + t])
