"""Helpers shared by the GPU parity tests (no arithmetic of the method lives here)."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_35140_b200 import synth

ATTN_TOL = 2e-2       # max-abs error of bf16 attention outputs against the fp64 oracle
LOGPROB_TOL = 5e-3    # max-abs error of fp32 log-probabilities against the fp64 oracle


def bits(t: torch.Tensor) -> torch.Tensor:
    """Reinterpret a bf16 / fp32 tensor as integers for exact comparison."""
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16)
    if t.dtype == torch.float32:
        return t.contiguous().view(torch.int32)
    raise TypeError(t.dtype)


def count_diff(a: torch.Tensor, b: torch.Tensor) -> int:
    return int((bits(a) != bits(b)).sum().item())


def canary_like(t: torch.Tensor, value: float = -777.0) -> torch.Tensor:
    return torch.full_like(t, value)


class Rollout:
    """Drives prefill + step-by-step decode of a workload through the library,
    writing K/V into a paged cache with the library's own cache-write."""

    def __init__(self, tik, w: synth.Workload, q, k, v, layout: synth.PagedLayout, dirty: float = 0.0):
        self.tik, self.w, self.q, self.k, self.v, self.layout = tik, w, q, k, v, layout
        dev = q.device
        self.dev = dev
        self.cu = w.cu_seqlens()
        self.bt = torch.from_numpy(layout.block_table).to(dev)
        shape = (layout.num_pages, w.Hkv, layout.page_size, w.d)
        self.kc = torch.full(shape, dirty, dtype=torch.bfloat16, device=dev)
        self.vc = torch.full(shape, dirty, dtype=torch.bfloat16, device=dev)
        self.scale = w.softmax_scale

    def _idx(self, ranges):
        return torch.cat([torch.arange(a, b, device=self.dev) for a, b in ranges])

    def prefill(self, seqs=None, start=None, stop=None):
        """Prefill positions [start[s], stop[s]) of the given sequences (default: whole prompts)."""
        w = self.w
        seqs = list(range(w.S)) if seqs is None else seqs
        start = [0] * len(seqs) if start is None else start
        stop = [w.prompt_lens[s] for s in seqs] if stop is None else stop
        rows = self._idx([(int(self.cu[s]) + a, int(self.cu[s]) + b) for s, a, b in zip(seqs, start, stop)])
        lens = [b - a for a, b in zip(start, stop)]
        cu_q = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=self.dev)
        ctx = torch.tensor(stop, dtype=torch.int32, device=self.dev)
        bt = self.bt[seqs].contiguous()
        self.tik.tik_kv_cache_write(self.k[rows].contiguous(), self.v[rows].contiguous(), cu_q, ctx,
                                    self.kc, self.vc, bt)
        o = self.tik.tik_attn_prefill(self.q[rows].contiguous(), cu_q, ctx, self.kc, self.vc, bt,
                                      max(lens), max(stop), self.scale)
        return rows, o

    def decode_step(self, seqs, positions, max_ctx=None, ws=None):
        """One decode step: sequence seqs[i] processes the token at positions[i]."""
        rows = torch.tensor([int(self.cu[s]) + p for s, p in zip(seqs, positions)], device=self.dev)
        B = len(seqs)
        cu1 = torch.arange(B + 1, dtype=torch.int32, device=self.dev)
        ctx = torch.tensor([p + 1 for p in positions], dtype=torch.int32, device=self.dev)
        bt = self.bt[seqs].contiguous()
        self.tik.tik_kv_cache_write(self.k[rows].contiguous(), self.v[rows].contiguous(), cu1, ctx,
                                    self.kc, self.vc, bt)
        mc = max(positions) + 1 if max_ctx is None else max_ctx
        o = self.tik.tik_attn_decode(self.q[rows].contiguous(), ctx, self.kc, self.vc, bt, mc,
                                     self.scale, ws=ws)
        return rows, o

    def replay(self):
        """Prefill all prompts, then decode every response token; returns o for all rows."""
        w = self.w
        out = torch.zeros_like(self.q)
        rows, o = self.prefill()
        out[rows] = o
        maxr = max(w.response_lens)
        for step in range(maxr):
            seqs = [s for s in range(w.S) if step < w.response_lens[s]]
            pos = [w.prompt_lens[s] + step for s in seqs]
            rows, o = self.decode_step(seqs, pos)
            out[rows] = o
        return out
