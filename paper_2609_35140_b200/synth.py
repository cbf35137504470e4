"""Seeded synthetic inputs shaped like the paper's RL workloads.

This module only draws random numbers and lays data out (packing, paging);
it contains none of the attention or log-probability arithmetic.  Both the
CUDA tests and the CPU-oracle tests take their inputs from here so that the
two implementations always see the same data.

The five workloads stand in for the prompt/response batches the paper trains
on (grade-school-math prompts answered by 1.5B-32B class models): only the
shapes, length mixes and value distributions are reproduced, never dataset
items.  Lengths come from numpy's default_rng, tensors from torch.Generator,
both seeded with 35140*10 + workload index.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import numpy as np
import torch

SEED_BASE = 35140 * 10


@dataclasses.dataclass
class Workload:
    index: int
    name: str
    Hq: int
    Hkv: int
    d: int
    page_size: int
    prompt_lens: List[int]          # per sequence
    response_lens: List[int]        # per sequence
    group_of: List[int]             # sequences with the same group share their prompt
    hidden: int
    vocab: int
    decode_contexts: Optional[List[int]] = None   # timed decode contexts (workload 3 only)

    @property
    def S(self) -> int:
        return len(self.prompt_lens)

    @property
    def seq_lens(self) -> List[int]:
        return [p + r for p, r in zip(self.prompt_lens, self.response_lens)]

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def response_tokens(self) -> int:
        return int(sum(self.response_lens))

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def seed(self) -> int:
        return SEED_BASE + self.index

    @property
    def softmax_scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.d)))

    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seq_lens)]).astype(np.int32)

    def causal_pairs(self) -> int:
        return int(sum(L * (L + 1) // 2 for L in self.seq_lens))

    def train_flops(self) -> float:
        """Algorithmic flops of the packed causal forward: QK^T and PV over causal pairs."""
        return 4.0 * self.d * self.Hq * self.causal_pairs()

    def prefill_flops(self) -> float:
        seen = set()
        pairs = 0
        for p, g in zip(self.prompt_lens, self.group_of):
            if g in seen:
                continue
            seen.add(g)
            pairs += p * (p + 1) // 2
        return 4.0 * self.d * self.Hq * pairs

    def logprob_flops(self, T: Optional[int] = None) -> float:
        T = self.response_tokens if T is None else T
        return 2.0 * T * self.hidden * self.vocab


def _uniform_int(rng, lo, hi, n):
    return [int(x) for x in rng.integers(lo, hi + 1, size=n)]


def get_workload(index: int) -> Workload:
    """The five benchmark workloads (index 0..4)."""
    rng = np.random.default_rng(SEED_BASE + index)
    if index == 0:
        return Workload(0, "tiny", 4, 1, 64, 16, [64, 64], [32, 96], [0, 1], 256, 2048)
    if index == 1:
        S = 16
        return Workload(1, "1.5B-class", 12, 2, 128, 64, [512] * S,
                        _uniform_int(rng, 128, 2048, S), list(range(S)), 1536, 151936)
    if index == 2:
        groups, per = 8, 8
        S = groups * per
        return Workload(2, "7B-GRPO", 28, 4, 128, 64, [1024] * S,
                        _uniform_int(rng, 256, 4096, S), [i // per for i in range(S)],
                        3584, 152064)
    if index == 3:
        S = 16
        return Workload(3, "long-context", 32, 8, 128, 64, [2048] * S, [14336] * S,
                        list(range(S)), 4096, 151936, decode_contexts=[4096, 8192, 16384])
    if index == 4:
        S = 256
        sigma = 0.8
        mu = math.log(2048.0) - 0.5 * sigma * sigma
        r = np.rint(rng.lognormal(mu, sigma, size=S)).astype(np.int64)
        r = np.clip(r, 16, 8192)
        return Workload(4, "32B-large-batch", 64, 8, 128, 64, [1024] * S,
                        [int(x) for x in r], list(range(S)), 5120, 151936)
    raise ValueError("workload index must be 0..4")


def custom_workload(prompt_lens, response_lens, Hq, Hkv, d, page_size, hidden=256, vocab=2048,
                    group_of=None, index=99) -> Workload:
    S = len(prompt_lens)
    return Workload(index, "custom", Hq, Hkv, d, page_size, list(prompt_lens),
                    list(response_lens), list(group_of) if group_of else list(range(S)),
                    hidden, vocab)


def _randn_bf16(shape, gen, device, std=1.0, chunk_rows=1 << 16):
    """N(0, std) in fp32 rounded to bf16 (round-to-nearest-even), filled in row chunks."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    rows = shape[0]
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        blk = torch.randn((r1 - r0,) + tuple(shape[1:]), generator=gen, device=device,
                          dtype=torch.float32)
        if std != 1.0:
            blk *= std
        out[r0:r1] = blk.to(torch.bfloat16)
    return out


def make_qkv(w: Workload, device="cpu", seed_offset: int = 0) -> Tuple[
        torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]:
    """Packed q [tot,Hq,d], k, v [tot,Hkv,d] (bf16) and cu_seqlens (int32).

    Sequences of one group carry identical prompt rows (a shared prompt)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed + seed_offset)
    tot = w.total_tokens
    q = _randn_bf16((tot, w.Hq, w.d), gen, device)
    k = _randn_bf16((tot, w.Hkv, w.d), gen, device)
    v = _randn_bf16((tot, w.Hkv, w.d), gen, device)
    cu = w.cu_seqlens()
    first_of_group = {}
    for s, g in enumerate(w.group_of):
        if g not in first_of_group:
            first_of_group[g] = s
            continue
        src = int(cu[first_of_group[g]])
        dst = int(cu[s])
        P = w.prompt_lens[s]
        q[dst:dst + P] = q[src:src + P]
        k[dst:dst + P] = k[src:src + P]
        v[dst:dst + P] = v[src:src + P]
    return q, k, v, torch.from_numpy(cu).to(device)


@dataclasses.dataclass
class PagedLayout:
    """Physical placement of every sequence's logical pages."""
    page_size: int
    num_pages: int
    max_blocks: int
    block_table: np.ndarray         # int32 [S, max_blocks], -1 where unused
    shared_prompt_pages: int        # physical pages referenced by more than one sequence


def make_paged_layout(w: Workload, shuffle: bool = True, extra_pages: int = 3,
                      share_prompts: bool = True, page_size: Optional[int] = None) -> PagedLayout:
    """Assign physical pages: a seeded permutation of the pool (fragmented placement);
    sequences of one group point at the same physical pages for their full prompt pages."""
    page = page_size or w.page_size
    rng = np.random.default_rng(w.seed + 7919)
    nblk = [(L + page - 1) // page for L in w.seq_lens]
    max_blocks = max(nblk)
    need = 0
    owner_pages = {}
    plan = []
    for s, g in enumerate(w.group_of):
        shared = 0
        if share_prompts and g in owner_pages:
            shared = w.prompt_lens[s] // page      # whole prompt pages only
        else:
            owner_pages[g] = s
        plan.append((s, g, shared))
        need += nblk[s] - shared
    num_pages = need + extra_pages
    perm = rng.permutation(num_pages) if shuffle else np.arange(num_pages)
    bt = -np.ones((w.S, max_blocks), dtype=np.int32)
    nxt = 0
    nshared = 0
    for s, g, shared in plan:
        if shared:
            bt[s, :shared] = bt[owner_pages[g], :shared]
            nshared += shared
        for b in range(shared, nblk[s]):
            bt[s, b] = perm[nxt]
            nxt += 1
    return PagedLayout(page, num_pages, max_blocks, bt, nshared)


def fill_paged_cache(w: Workload, layout: PagedLayout, k: torch.Tensor, v: torch.Tensor,
                     upto: Optional[List[int]] = None, fill: float = 0.0):
    """Scatter packed k/v rows into caches [num_pages,Hkv,page,d] (a pure copy).

    ``upto[s]`` limits how many tokens of sequence s are written (default: all)."""
    dev = k.device
    page = layout.page_size
    kc = torch.full((layout.num_pages, w.Hkv, page, w.d), fill, dtype=k.dtype, device=dev)
    vc = torch.full_like(kc, fill)
    cu = w.cu_seqlens()
    for s in range(w.S):
        n = w.seq_lens[s] if upto is None else int(upto[s])
        if n <= 0:
            continue
        pos = torch.arange(n, device=dev)
        phys = torch.from_numpy(layout.block_table[s]).to(dev)[pos // page].long()
        row = pos % page
        src = slice(int(cu[s]), int(cu[s]) + n)
        kc[phys, :, row, :] = k[src]
        vc[phys, :, row, :] = v[src]
    return kc, vc


def make_logprob_inputs(w: Workload, device="cpu", T: Optional[int] = None, seed_offset: int = 0):
    """hidden [T,H] ~ N(0,1), lm_head [V,H] ~ N(0, 0.02) (bf16), target ids uniform (int32)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed + 104729 + seed_offset)
    T = w.response_tokens if T is None else T
    hidden = _randn_bf16((T, w.hidden), gen, device)
    W = _randn_bf16((w.vocab, w.hidden), gen, device, std=0.02, chunk_rows=1 << 14)
    target = torch.randint(0, w.vocab, (T,), generator=gen, device=device, dtype=torch.int64)
    return hidden, W, target.to(torch.int32)


def make_rope_table(max_pos: int, d: int, base: float = 1.0e6, device="cpu") -> torch.Tensor:
    """The cos/sin table the pre-attention step takes as an input: fp32 [max_pos, d], row p =
    cos(p * theta_i) for i < d/2, then sin(p * theta_i), with theta_i = base^(-2i/d) (angles in fp64,
    rounded once).  base 1e6 is the Qwen2.5 / Qwen3 setting."""
    i = torch.arange(d // 2, dtype=torch.float64)
    theta = torch.pow(torch.tensor(float(base), dtype=torch.float64), -2.0 * i / d)
    ang = torch.arange(max_pos, dtype=torch.float64)[:, None] * theta[None, :]
    return torch.cat([torch.cos(ang), torch.sin(ang)], dim=1).to(torch.float32).to(device)


def make_norm_weights(w: Workload, device="cpu", seed_offset: int = 0):
    """Per-head RMSNorm weights for Q and K, bf16 [d] each, around one (trained norm weights
    stay close to their initial value of one)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed + 7919 + seed_offset)
    wq = (1.0 + 0.2 * torch.randn(w.d, generator=gen)).to(torch.bfloat16).to(device)
    wk = (1.0 + 0.2 * torch.randn(w.d, generator=gen)).to(torch.bfloat16).to(device)
    return wq, wk


def sample_rows(w: Workload, n_random: int, seed_offset: int = 1) -> List[Tuple[int, int, int]]:
    """(sequence, query head, position) rows worth checking one by one: every
    sequence's first and last row, rows around the 128-key tile, page and
    2048-key chunk boundaries, plus uniformly random rows."""
    rng = np.random.default_rng(w.seed + 31 * seed_offset)
    rows = set()
    for s, L in enumerate(w.seq_lens):
        marks = [0, L - 1, w.prompt_lens[s] - 1, w.prompt_lens[s]]
        for b in (w.page_size, 128, 2048):
            for m in range(b, L, b * max(1, (L // b) // 3)):
                marks += [m - 1, m, m + 1]
        for t in marks:
            if 0 <= t < L:
                rows.add((s, int(rng.integers(0, w.Hq)), int(t)))
    for _ in range(n_random):
        s = int(rng.integers(0, w.S))
        rows.add((s, int(rng.integers(0, w.Hq)), int(rng.integers(0, w.seq_lens[s]))))
    return sorted(rows)
