#!/usr/bin/env python
"""Benchmark of the unified attention + token log-prob hot path on B200.

One step = one pass of the whole hot path over one synthetic workload:
  train-forward attention over all packed sequences
  -> KV-cache write + prefill attention over the prompts
  -> one decode step (attention + split-KV combine) per timed context
  -> token log-probabilities over all response tokens.
Headline metric: summed train-forward + prefill + decode attention time (ms, lower is
better) on the largest workload, configs[4]; decode tokens/s, the log-prob time and
per-kernel roofline fractions ride along.

With no --workload the run covers all five workloads: configs[0..3] first (a few steps each,
reported under `per_config`), then configs[4] with exactly --warmup untimed and --steps timed
steps: that is the timed region of the JSON line (`value`, `ms_per_step`, `roofline`, `clocks`).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--impl tik|reference]

N > 1 (torchrun, one rank per GPU): N independent replicas, no collective on the data path;
the reported times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_35140_b200 import dist as tdist  # noqa: E402
from paper_2609_35140_b200 import synth  # noqa: E402
from paper_2609_35140_b200.microbench import L2Flush  # noqa: E402

METRIC = "summed_attention_ms"
HEADLINE = 4                      # configs[4], the largest single-GPU workload
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 7700.0}     # data-sheet figures, context only
SM_COUNT, MMA_FLOP_PER_CLK_SM = 148, 8192                 # M128 N128 K16 bf16 MMA: 64 clk
# DRAM bytes per launch of the headline's dominant kernel (attn_kernel<128, train>) from ncu:
# captured on a slice of the workload and scaled by tokens (see profiles/), None until captured.
NCU_TRAFFIC = {"bytes_per_token": 39225.0,
               "source": "ncu dram__bytes_read+write of attn_persist_kernel<128,packed> on the first 32 sequences of this "
                         "workload (3.93 GB for 100 313 tokens, 1.06 x the algorithmic q+k+v+o), scaled by tokens: "
                         "profiles/attention_fullseq_judged_sizes.md"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return {k: float(pk[k]) for k in FALLBACK_PEAKS if k in pk}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period, self.stop_flag = index, period_s, threading.Event()
        self.sm, self.reasons, self.max_sm, self.ok = [], set(), None, False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self.stop_flag.is_set():
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self.stop_flag.set()
        self.join()
        if not self.ok or not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.sm)), "sm_mhz_min": float(np.min(self.sm)), "sm_max_mhz": self.max_sm,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------
class HotPath:
    """Device-resident inputs of one workload replica and the calls of one step."""

    def __init__(self, tik, w: synth.Workload, seed_offset: int = 0):
        self.tik, self.w = tik, w
        dev = "cuda"
        self.q, self.k, self.v, self.cu = synth.make_qkv(w, dev, seed_offset)
        self.layout = synth.make_paged_layout(w)
        self.bt = torch.from_numpy(self.layout.block_table).to(dev)
        shape = (self.layout.num_pages, w.Hkv, self.layout.page_size, w.d)
        self.kc = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
        self.vc = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
        cu_h = w.cu_seqlens()
        self.cu_h = cu_h
        # whole cache resident (decode at full context reads it)
        ctx_full = torch.tensor(w.seq_lens, dtype=torch.int32, device=dev)
        tik.tik_kv_cache_write(self.k, self.v, self.cu, ctx_full, self.kc, self.vc, self.bt)
        # prefill: one prompt per group (sequences of a group share prompt pages)
        firsts = []
        seen = set()
        for s, g in enumerate(w.group_of):
            if g not in seen:
                seen.add(g)
                firsts.append(s)
        self.pre_seqs = firsts
        rows = torch.cat([torch.arange(cu_h[s], cu_h[s] + w.prompt_lens[s]) for s in firsts]).to(dev)
        self.pre_q = self.q[rows].contiguous()
        self.pre_k = self.k[rows].contiguous()
        self.pre_v = self.v[rows].contiguous()
        plens = [w.prompt_lens[s] for s in firsts]
        self.pre_cu = torch.tensor(np.concatenate([[0], np.cumsum(plens)]), dtype=torch.int32, device=dev)
        self.pre_ctx = torch.tensor(plens, dtype=torch.int32, device=dev)
        self.pre_bt = self.bt[firsts].contiguous()
        self.pre_max = max(plens)
        self.pre_o = torch.empty_like(self.pre_q)
        # decode points: full context of every sequence, or the listed contexts
        self.dec = []
        ctxs = w.decode_contexts or [None]
        for c in ctxs:
            lens = [min(L, c) if c else L for L in w.seq_lens]
            rows = torch.tensor([cu_h[s] + lens[s] - 1 for s in range(w.S)]).to(dev)
            self.dec.append({
                "ctx": torch.tensor(lens, dtype=torch.int32, device=dev), "max": max(lens),
                "q": self.q[rows].contiguous(), "o": torch.empty(w.S, w.Hq, w.d, dtype=torch.bfloat16, device=dev),
                "bytes": self._decode_bytes(lens), "logical_bytes": sum(lens) * w.Hkv * w.d * 2 * 2,
                "label": c or "full"})
        need = max(tik.workspace_bytes(tik.OP_ATTN_DECODE, w.S, w.Hq, w.Hkv, w.d, d["max"]) for d in self.dec)
        self.dec_ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
        self.o = torch.empty_like(self.q)
        # log-prob over all response tokens
        self.hidden, self.W, self.target = synth.make_logprob_inputs(w, dev, seed_offset=seed_offset)
        self.lp = torch.empty(self.hidden.shape[0], dtype=torch.float32, device=dev)
        need = tik.workspace_bytes(tik.OP_TOKEN_LOGPROB, self.hidden.shape[0], H=w.hidden, V=w.vocab)
        self.lp_ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
        self.flush = L2Flush(dev)      # 512 MiB written, then 256 MiB read: cold AND clean L2 before a phase
        # train 1; cache write + prefill 2; decode + combine per point; log-prob + finish 2
        self.launches_per_step = 1 + 2 + 2 * len(self.dec) + 2     # entry-point calls' minimum; the library counts the real launches
        self.launches_in_timed_region = 0

    def _decode_bytes(self, lens):
        """Unique K+V bytes one decode step must read (shared prompt pages counted once)."""
        w, page = self.w, self.layout.page_size
        pages = set()
        partial = 0
        for s, L in enumerate(lens):
            full = L // page
            for b in range(full):
                pages.add(int(self.layout.block_table[s, b]))
            partial += L - full * page
        return (len(pages) * page + partial) * w.Hkv * w.d * 2 * 2

    # -- single phases
    def train(self, q=None, k=None, v=None, cu=None, o=None):
        w = self.w
        self.tik.tik_attn_train_fwd(self.q if q is None else q, self.k if k is None else k, self.v if v is None else v,
                                    self.cu if cu is None else cu, max(w.seq_lens), w.softmax_scale,
                                    o=self.o if o is None else o)

    def prefill(self, pq=None, pk=None, pv=None, o=None):
        tik, w = self.tik, self.w
        tik.tik_kv_cache_write(self.pre_k if pk is None else pk, self.pre_v if pv is None else pv, self.pre_cu,
                               self.pre_ctx, self.kc, self.vc, self.pre_bt)
        tik.tik_attn_prefill(self.pre_q if pq is None else pq, self.pre_cu, self.pre_ctx, self.kc, self.vc, self.pre_bt,
                             self.pre_max, self.pre_max, w.softmax_scale, o=self.pre_o if o is None else o)

    def decode(self, i, q=None, o=None):
        d = self.dec[i]
        self.tik.tik_attn_decode(d["q"] if q is None else q, d["ctx"], self.kc, self.vc, self.bt, d["max"],
                                 self.w.softmax_scale, ws=self.dec_ws, o=d["o"] if o is None else o)

    def logprob(self):
        self.tik.tik_token_logprob(self.hidden, self.W, self.target, ws=self.lp_ws, logprob=self.lp)

    # -- the calls of one step; `mark(name)` records an event after each phase
    def step(self, mark, flush=True):
        def fl(name):
            if flush:
                self.flush.zero_()
            mark(name)
        fl("flush0")
        self.train()
        mark("train")
        fl("flush1")
        self.prefill()
        mark("prefill")
        for i in range(len(self.dec)):
            fl("flushd%d" % i)
            self.decode(i)
            mark("decode%d" % i)
        fl("flush2")
        self.logprob()
        mark("logprob")


def time_steps(hp: HotPath, steps: int, warmup: int):
    """Returns (per-phase mean ms, total ms per step) measured with CUDA events."""
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        hp.step(lambda name: None)
    torch.cuda.synchronize()
    tdist.barrier()
    torch.cuda.synchronize()
    events = []
    launches0 = hp.tik.kernel_launches()
    start = torch.cuda.Event(enable_timing=True)
    start.record(stream)
    for _ in range(steps):
        evs = []

        def mark(name, evs=evs):
            e = torch.cuda.Event(enable_timing=True)
            e.record(stream)
            evs.append((name, e))
        hp.step(mark)
        events.append(evs)
    end = torch.cuda.Event(enable_timing=True)
    end.record(stream)
    hp.launches_in_timed_region = hp.tik.kernel_launches() - launches0      # the library's own count
    torch.cuda.synchronize()
    tdist.barrier()
    total_ms = start.elapsed_time(end) / steps
    phase = {}
    for evs in events:
        prev = None
        for name, e in evs:
            if prev is not None and not name.startswith("flush"):
                phase[name] = phase.get(name, 0.0) + prev.elapsed_time(e)
            prev = e
    phase = {k: v / steps for k, v in phase.items()}
    return phase, total_ms


ALONE_PAUSE_S = 1.0      # idle time between the timed steps and the phases timed on their own


def time_alone(hp: HotPath, fn, reps: int, warmup: int = 2):
    """Median ms of `fn` launched on its own: (L2 flush, event, fn, event) x reps queued back to
    back and synchronised once, so the host's share of a call hides behind the previous flush.
    Calls shorter than a millisecond are repeated until there are 20 readings."""
    def batch(n):
        evs = []
        for _ in range(n):
            hp.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    ts = sorted(batch(warmup + reps)[warmup:])
    if ts[len(ts) // 2] < 1.0 and len(ts) < 20:
        ts = sorted(ts + batch(20 - len(ts)))
    return ts[len(ts) // 2]


def time_decode_graph(hp: HotPath, i: int, nsteps: int = 20):
    """One decode point as a CUDA graph of `nsteps` identical steps (each: L2 flush, decode, combine),
    replayed three times; the time of a graph of `nsteps` flushes alone is taken off.  Returns ms per
    step, or None with the reason when the calls cannot be captured."""
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):                 # everything the capture needs has run once
            hp.flush.zero_()
            hp.decode(i)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g_all, g_flush = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_all):
            for _ in range(nsteps):
                hp.flush.zero_()
                hp.decode(i)
        with torch.cuda.graph(g_flush):
            for _ in range(nsteps):
                hp.flush.zero_()
        ts = []
        for g in (g_all, g_flush):
            best = None
            for _ in range(4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                g.replay()
                e1.record()
                torch.cuda.synchronize()
                t = e0.elapsed_time(e1)
                best = t if best is None else min(best, t)
            ts.append(best)
        del g_all, g_flush
        return max(ts[0] - ts[1], 0.0) / nsteps, None
    except Exception as exc:     # capture is an extra: the eager numbers stand without it
        torch.cuda.synchronize()
        return None, "%s: %s" % (type(exc).__name__, str(exc)[:200])


# ------------------------------------------------------------------------------------------ end to end
class PinnedRing:
    """A bounded ring of pinned host slots through which tensors of any size cross PCIe: a slice
    is staged from pageable host memory into a free slot and copied on with one asynchronous
    copy (host -> device), or copied into a free slot (device -> host).  A slot is reused once
    the copy that last used it has completed."""

    def __init__(self, slot_bytes: int = 128 << 20, nslots: int = 8):
        self.slot_bytes = slot_bytes
        self.slots = [torch.empty(slot_bytes, dtype=torch.uint8).pin_memory() for _ in range(nslots)]
        self.busy = [None] * nslots
        self.i = 0

    @property
    def pinned_bytes(self):
        return self.slot_bytes * len(self.slots)

    def _slot(self):
        k = self.i % len(self.slots)
        self.i += 1
        if self.busy[k] is not None:
            self.busy[k].synchronize()
        return k

    def h2d(self, dst: torch.Tensor, src: torch.Tensor, stream) -> int:
        d = dst.reshape(-1).view(torch.uint8)
        s = src.reshape(-1).view(torch.uint8)
        n = d.numel()
        for off in range(0, n, self.slot_bytes):
            m = min(self.slot_bytes, n - off)
            k = self._slot()
            self.slots[k][:m].copy_(s[off:off + m])                      # pageable -> pinned
            with torch.cuda.stream(stream):
                d[off:off + m].copy_(self.slots[k][:m], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(stream)
            self.busy[k] = ev
        return n

    def d2h(self, src: torch.Tensor, stream) -> int:
        s = src.reshape(-1).view(torch.uint8)
        n = s.numel()
        for off in range(0, n, self.slot_bytes):
            m = min(self.slot_bytes, n - off)
            k = self._slot()
            with torch.cuda.stream(stream):
                self.slots[k][:m].copy_(s[off:off + m], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(stream)
            self.busy[k] = ev
        return n


def time_e2e(hp: HotPath, steps: int, warmup: int):
    """Attention phases end to end through the public API: every step brings its inputs in from the
    host and takes its outputs back, both through bounded rings of pinned slots (1 GiB each) with one
    asynchronous copy per slice.  Three streams and two sets of device buffers: the copy-in of step
    s+1 and the copy-out of step s-1 run under the kernels of step s.  Timed from the first copy-in
    to the last copy-out."""
    comp = torch.cuda.current_stream()
    names = ("q", "k", "v", "pre_q", "pre_k", "pre_v")
    host_in = {n: getattr(hp, n).cpu() for n in names}
    host_in.update({"dq%d" % i: d["q"].cpu() for i, d in enumerate(hp.dec)})
    dev_in = [{n: torch.empty(t.shape, dtype=t.dtype, device="cuda") for n, t in host_in.items()} for _ in range(2)]
    dev_out = [{"o": torch.empty_like(hp.o), "pre_o": torch.empty_like(hp.pre_o),
                **{"do%d" % i: torch.empty_like(d["o"]) for i, d in enumerate(hp.dec)}} for _ in range(2)]
    ring_in, ring_out = PinnedRing(), PinnedRing()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    in_done = [torch.cuda.Event() for _ in range(2)]
    comp_done = [torch.cuda.Event() for _ in range(2)]
    out_done = [torch.cuda.Event() for _ in range(2)]
    counts = {"h2d": 0, "d2h": 0}

    def run(n_steps, t0=None, t1=None):
        for s in range(n_steps):
            b = s & 1
            if s == 0 and t0 is not None:
                t0.record(s_in)
            if s >= 2:
                s_in.wait_event(comp_done[b])                # step s-2 has consumed this input set
            h = 0
            for n, t in host_in.items():
                h += ring_in.h2d(dev_in[b][n], t, s_in)
            in_done[b].record(s_in)
            comp.wait_event(in_done[b])
            if s >= 2:
                comp.wait_event(out_done[b])                 # step s-2's outputs have left this output set
            di, do = dev_in[b], dev_out[b]
            hp.train(di["q"], di["k"], di["v"], hp.cu, do["o"])
            hp.prefill(di["pre_q"], di["pre_k"], di["pre_v"], do["pre_o"])
            for i in range(len(hp.dec)):
                hp.decode(i, di["dq%d" % i], do["do%d" % i])
            comp_done[b].record(comp)
            s_out.wait_event(comp_done[b])
            g = 0
            for n, t in do.items():
                g += ring_out.d2h(t, s_out)
            out_done[b].record(s_out)
            counts["h2d"], counts["d2h"] = h, g
            if s == n_steps - 1 and t1 is not None:
                t1.record(s_out)

    run(max(2, warmup))
    torch.cuda.synchronize()
    tdist.barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    run(steps, t0, t1)
    torch.cuda.synchronize()
    tdist.barrier()
    return t0.elapsed_time(t1) / steps, counts["h2d"], counts["d2h"], ring_in.pinned_bytes + ring_out.pinned_bytes


# ------------------------------------------------------------------------------------------ rollout replay
def time_replay(hp: HotPath):
    """The whole rollout for real: cache write + prefill of the prompts, then every decode step
    (cache write of the step's tokens, decode attention, combine) until the longest response ends,
    the batch shrinking as sequences finish.  Response tokens are laid out step-major beforehand so
    that a step's rows are one contiguous slice.  Returns (total ms, decode steps, launches)."""
    tik, w = hp.tik, hp.w
    dev = "cuda"
    order = sorted(range(w.S), key=lambda s: -w.response_lens[s])
    R = [w.response_lens[s] for s in order]
    P = [w.prompt_lens[s] for s in order]
    nsteps = R[0]
    active = [sum(1 for r in R if r > t) for t in range(nsteps)]
    idx = np.concatenate([[hp.cu_h[order[i]] + P[i] + t for i in range(active[t])] for t in range(nsteps)]).astype(np.int64)
    idx_d = torch.from_numpy(idx).to(dev)
    q_sm, k_sm, v_sm = hp.q[idx_d], hp.k[idx_d], hp.v[idx_d]
    o_sm = torch.empty_like(q_sm)
    off = np.concatenate([[0], np.cumsum(active)]).astype(np.int64)
    bt = hp.bt[order].contiguous()
    ctx_all = (torch.tensor(P, dtype=torch.int32)[None, :] + torch.arange(1, nsteps + 1, dtype=torch.int32)[:, None]).to(dev)
    cu1 = torch.arange(w.S + 1, dtype=torch.int32, device=dev)
    max_ctx = [max(P[:active[t]]) + t + 1 for t in range(nsteps)]
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    hp.flush.zero_()
    e0.record()
    hp.prefill()
    for t in range(nsteps):
        n, a, b = active[t], int(off[t]), int(off[t + 1])
        ctx = ctx_all[t, :n]
        btn = bt[:n]
        tik.tik_kv_cache_write(k_sm[a:b], v_sm[a:b], cu1[:n + 1], ctx, hp.kc, hp.vc, btn)
        tik.tik_attn_decode(q_sm[a:b], ctx, hp.kc, hp.vc, btn, max_ctx[t], w.softmax_scale, ws=hp.dec_ws, o=o_sm[a:b])
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), nsteps, 2 + 3 * nsteps


# ------------------------------------------------------------------------------------------ beside the step
def time_prep(hp: "HotPath", reps: int = 5):
    """The pre-attention step (per-head RMSNorm -> NeoX RoPE -> paged cache write) over all tokens of
    the workload, measured on its own after the timed steps: it widens the path beyond the metric's
    step, so it is reported beside it, not inside it.  Returns (median ms, algorithmic bytes)."""
    tik, w = hp.tik, hp.w
    q, k = hp.q.clone(), hp.k.clone()
    kc, vc = torch.zeros_like(hp.kc), torch.zeros_like(hp.vc)
    wq, wk = synth.make_norm_weights(w, "cuda")
    tab = synth.make_rope_table(max(w.seq_lens), w.d, device="cuda")
    ctx = torch.tensor(w.seq_lens, dtype=torch.int32, device="cuda")
    ms = time_alone(hp, lambda: tik.tik_qk_norm_rope_kv_write(q, k, hp.v, wq, wk, 1e-6, tab, hp.cu, ctx, kc, vc, hp.bt), reps)
    # per token: q and k read and written, v read, K and V cache rows written, one table row read
    byt = w.total_tokens * ((w.Hq + w.Hkv) * w.d * 2 * 2 + 3 * w.Hkv * w.d * 2 + w.d * 4)
    return ms, byt


def time_bwd(hp: "HotPath", burst, reps: int = 3):
    """The policy-update backward of the train-forward phase (dQ, dK, dV), timed on its own."""
    tik, w = hp.tik, hp.w
    gen = torch.Generator(device="cuda").manual_seed(w.seed + 777)
    do = synth._randn_bf16(tuple(hp.q.shape), gen, "cuda")
    lse = torch.empty(hp.q.shape[0], w.Hq, dtype=torch.float32, device="cuda")
    o = tik.tik_attn_train_fwd(hp.q, hp.k, hp.v, hp.cu, max(w.seq_lens), w.softmax_scale, lse=lse)
    ws = torch.empty(max(16, tik.workspace_bytes(tik.OP_ATTN_TRAIN_BWD, hp.q.shape[0], w.Hq, w.Hkv, w.d)),
                     dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    time.sleep(ALONE_PAUSE_S)
    ms = time_alone(hp, lambda: tik.tik_attn_train_bwd(hp.q, hp.k, hp.v, o, do, lse, hp.cu, max(w.seq_lens),
                                                        w.softmax_scale, ws=ws), reps, warmup=1)
    tf = 2.5 * w.train_flops() / (ms * 1e-3) / 1e12
    return {"bound": "tensor", "achieved": tf, "peak": burst, "unit": "TFLOP/s", "frac": tf / burst, "ms": ms,
            "note": "algorithmic flops = 2.5 x the forward's (five products against two); the two-pass kernel "
                    "executes 3.5 x; beside the step, not part of the metric"}


FFN_INTERMEDIATE = {256: 704, 1536: 8960, 3584: 18944, 4096: 12288, 5120: 27648}   # Qwen2.5 / Qwen3 class shapes


def time_ffn(hp: "HotPath", peaks, tpeak, reps: int = 5):
    """The FFN-side operators (hidden RMSNorm, fused residual + RMSNorm, gate/up projection, SwiGLU,
    down projection) on up to 32 768 tokens of the workload's hidden size, each timed on its own
    with an L2 flush before every launch.  Reported beside the step, not part of the metric."""
    tik, w = hp.tik, hp.w
    T, H = min(w.total_tokens, 32768), w.hidden
    I = FFN_INTERMEDIATE.get(H, 4 * H)
    gen = torch.Generator(device="cuda").manual_seed(w.seed + 4242)

    def rn(shape, std=1.0):
        return (torch.randn(shape, generator=gen, device="cuda") * std).to(torch.bfloat16)

    x, res, wn = rn((T, H)), rn((T, H)), (1 + 0.1 * rn((H,)).float()).to(torch.bfloat16)
    w_gu, w_d = rn((2 * I, H), 0.02), rn((H, I), 0.02)
    h = torch.empty_like(x)
    gu = torch.empty(T, 2 * I, dtype=torch.bfloat16, device="cuda")
    act = torch.empty(T, I, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(x)

    def hbm(ms, byt, note):
        g = byt / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": g, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": g / peaks["hbm_gbs"],
                "ms": ms, "bytes": byt, "note": note}

    def tensor(ms, flops, note):
        tf = flops / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak, "ms": ms,
                "note": note}

    shape = "T=%d H=%d I=%d; beside the step, not part of the metric" % (T, H, I)
    # The HBM-bound operators first, after an idle second (the power state of what ran before has
    # decayed: they are bandwidth measurements), the two big GEMMs last; the order does not matter
    # for the values computed, only `gu` and `act` need finite contents before they are read.
    gu.normal_()
    act.normal_()
    xd, yd = x[:min(w.S, 256)].contiguous(), torch.empty(min(w.S, 256), 2 * I, dtype=torch.bfloat16, device="cuda")
    ad, od = act[:xd.shape[0]].contiguous(), torch.empty(xd.shape[0], H, dtype=torch.bfloat16, device="cuda")
    torch.cuda.synchronize()
    time.sleep(ALONE_PAUSE_S)
    r = {}
    r["rmsnorm"] = hbm(time_alone(hp, lambda: tik.tik_rmsnorm(x, wn, 1e-6, y=h), reps), 2 * T * H * 2, shape)
    r["add_rmsnorm"] = hbm(time_alone(hp, lambda: tik.tik_rmsnorm(x, wn, 1e-6, residual=res, y=h), reps), 4 * T * H * 2, shape)
    r["swiglu"] = hbm(time_alone(hp, lambda: tik.tik_swiglu(gu, out=act), reps), 3 * T * I * 2, shape)
    # decode-sized projections: one token per sequence, the weights are streamed once (HBM-bound)
    r["linear_gate_up_decode_shaped"] = hbm(time_alone(hp, lambda: tik.tik_linear(xd, w_gu, y=yd), reps), 2 * I * H * 2,
                                            "T=%d rows: weight bytes 2I*H*2 over the launch time%s" % (
                                                xd.shape[0], "; at 256 rows the call needs as long on the tensor pipes as on HBM "
                                                "(ridge point), so it follows the SM clock" if xd.shape[0] > 128 else ""))
    r["linear_down_decode_shaped"] = hbm(time_alone(hp, lambda: tik.tik_linear(ad, w_d, y=od), reps), I * H * 2,
                                         "T=%d rows: weight bytes I*H*2 over the launch time; the fixed K chain of "
                                         "I/16 MMAs per element on at most H/64 CTAs bounds it" % xd.shape[0])
    r["linear_gate_up"] = tensor(time_alone(hp, lambda: tik.tik_linear(h, w_gu, y=gu), reps), 2.0 * T * H * 2 * I, shape)
    r["linear_down"] = tensor(time_alone(hp, lambda: tik.tik_linear(act, w_d, y=out), reps), 2.0 * T * I * H, shape)
    return r


# ------------------------------------------------------------------------------------------
def oracle_sample_ms(w: synth.Workload, seed: int = 0, target_pairs: float = 2.5e8):
    """Times the CPU oracle on a bounded sample of the workload's attention rows and scales
    by causal (query, key) pairs to the summed-attention metric.  Returns
    (extrapolated ms, cores, description, measured seconds)."""
    import oracle
    rng = np.random.default_rng(w.seed + 555 + seed)
    # metric pairs: train rows + prefill rows + decode rows (per query head)
    firsts = {}
    for s, g in enumerate(w.group_of):
        firsts.setdefault(g, s)
    pre_pairs = sum(w.prompt_lens[s] * (w.prompt_lens[s] + 1) // 2 for s in firsts.values())
    ctxs = w.decode_contexts or [None]
    dec_pairs = sum(sum(min(L, c) if c else L for L in w.seq_lens) for c in ctxs)
    metric_pairs = (w.causal_pairs() + pre_pairs + dec_pairs) * w.Hq
    # one KV head's K/V for up to 32 sequences, then random (sequence, position) rows until the
    # sample holds about 2.5e8 query-key pairs (a few seconds on the machine's cores)
    gen = torch.Generator().manual_seed(w.seed + 99)
    pool = [int(s) for s in rng.permutation(w.S)[:32]]
    offs, lens, kparts, vparts, starts = [], [], [], [], {}
    base = 0
    for s in pool:
        L = w.seq_lens[s]
        kparts.append(torch.randn(L, w.d, generator=gen).to(torch.bfloat16).float().numpy())
        vparts.append(torch.randn(L, w.d, generator=gen).to(torch.bfloat16).float().numpy())
        starts[s] = base
        base += L
    pairs = 0
    while pairs < min(target_pairs, metric_pairs):
        s = pool[int(rng.integers(0, len(pool)))]
        t = int(rng.integers(0, w.seq_lens[s]))
        offs.append(starts[s])
        lens.append(t + 1)
        pairs += t + 1
    kflat, vflat = np.concatenate(kparts), np.concatenate(vparts)
    qrows = torch.randn(len(lens), w.d, generator=gen).to(torch.bfloat16).float().numpy()
    t0 = time.perf_counter()
    oracle.attn_rows(qrows, kflat, vflat, offs, lens, w.softmax_scale)
    dt = time.perf_counter() - t0
    ms = dt * 1e3 * (metric_pairs / max(pairs, 1))
    desc = ("oracle.attn_rows on %d sampled rows (%.3g of %.3g causal query-key pairs of train+prefill+decode), "
            "%.2f s measured, scaled by pairs" % (len(lens), pairs, metric_pairs, dt))
    return ms, oracle.num_threads(), desc, dt


def run_reference(args, rank, world):
    if rank != 0:
        return
    w = synth.get_workload(HEADLINE if args.workload is None else args.workload)
    vals = []
    desc, cores = "", 0
    for i in range(args.warmup + args.steps):
        ms, cores, desc, _ = oracle_sample_ms(w, seed=i, target_pairs=1.0e8)
        if i >= args.warmup:
            vals.append(ms)
    v = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "ms", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": v, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args.gpus),
            "cpu_baseline": {"value": v, "unit": "ms", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": v, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_config(w: synth.Workload, n_gpus: int):
    return {"workload": "configs[%d] %s" % (w.index, w.name), "sequences": w.S, "Hq": w.Hq, "Hkv": w.Hkv,
            "head_dim": w.d, "page_size": w.page_size, "total_tokens": w.total_tokens,
            "response_tokens": w.response_tokens, "hidden": w.hidden, "vocab": w.vocab,
            "decode_contexts": w.decode_contexts or "full sequence lengths",
            "l2": "before every phase a 512 MiB buffer is overwritten (L2 flush) and a 256 MiB buffer is read (pushes the "
                  "flush's own dirty lines out, so the phase does not pay for their write-back); excluded from the phase times",
            "alone": "the phases timed on their own follow the steps after %.0f s of idle time (the step's "
                     "power state has decayed); they are context for the in-step figures, not part of `value`" % ALONE_PAUSE_S,
            "parallelism": "replicas x%d (no collective)" % n_gpus}


# ------------------------------------------------------------------------------------------ one workload
def measure_workload(tik, w, steps, warmup, rank, local_rank, headline: bool, want_replay: bool):
    """Times one workload; returns (flat dict of numbers to be max-reduced over ranks, info dict)."""
    hp = HotPath(tik, w, seed_offset=tdist.replica_seed_offset(rank))
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    t_wall = time.perf_counter()
    phase, total_ms = time_steps(hp, steps, warmup)
    region_s = time.perf_counter() - t_wall
    clk = sampler.finish()
    nums = dict(phase)
    nums["total"] = total_ms
    # every attention phase once more on its own (short bursts: the clocks are not held down by the
    # log-prob GEMM of the same step), and the decode-shaped log-prob call (one row per sequence)
    reps = max(3, min(steps, 10))
    torch.cuda.synchronize()
    time.sleep(ALONE_PAUSE_S)          # the power state of the steps decays before the short bursts are timed
    nums["alone_train"] = time_alone(hp, hp.train, reps)
    nums["alone_prefill"] = time_alone(hp, hp.prefill, reps)
    for i in range(len(hp.dec)):
        nums["alone_decode%d" % i] = time_alone(hp, lambda i=i: hp.decode(i), reps)
    graph_notes = []
    for i in range(len(hp.dec)):
        ms_g, why = time_decode_graph(hp, i)
        nums["graph_decode%d" % i] = ms_g if ms_g is not None else -1.0
        graph_notes.append(why)
    nb = min(w.S, 256)
    hid_b, tgt_b = hp.hidden[:nb].contiguous(), hp.target[:nb].contiguous()
    lp_b = torch.empty(nb, dtype=torch.float32, device="cuda")
    nums["logprob_decode_shaped"] = time_alone(
        hp, lambda: tik.tik_token_logprob(hid_b, hp.W, tgt_b, ws=hp.lp_ws, logprob=lp_b), reps)
    info = {"clocks": clk, "region_s": region_s, "launches_per_step": hp.launches_per_step,
            "launches_timed": hp.launches_in_timed_region,
            "dec": [{"label": d["label"], "bytes": d["bytes"], "logical_bytes": d["logical_bytes"],
                     "graph_note": graph_notes[j]} for j, d in enumerate(hp.dec)], "lp_rows": nb}
    if want_replay:
        ms, nsteps, launches = time_replay(hp)
        nums["replay_total"] = ms
        info["replay"] = {"decode_steps": nsteps, "launches": launches}
    return hp, nums, info


def report_workload(w, nums, info, peaks, world):
    """Per-workload block of the JSON line: phase times, rates and roofline fractions."""
    burst, sust, hbm = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"], peaks["hbm_gbs"]
    clk = info["clocks"]
    mhz, mx = clk.get("sm_mhz"), clk.get("sm_max_mhz")

    def tensor(flops, ms, alone_ms=None):
        tf = flops / (ms * 1e-3) / 1e12
        r = {"ms": ms, "tflops": tf, "frac_burst_peak": tf / burst, "frac_sustained_peak": tf / sust,
             "frac_nominal_peak": tf / NOMINAL["bf16_tflops"]}
        if mhz:
            # what the tensor pipes could do at the clock the region actually ran at
            r["frac_of_pipe_rate_at_sampled_clock"] = tf * 1e12 / (SM_COUNT * MMA_FLOP_PER_CLK_SM * mhz * 1e6)
        if alone_ms is not None:
            ta = flops / (alone_ms * 1e-3) / 1e12
            r["alone"] = {"ms": alone_ms, "tflops": ta, "frac_burst_peak": ta / burst}
        return r

    dec_keys = sorted(k for k in nums if k.startswith("decode"))
    t_dec = [nums[k] for k in dec_keys]
    out = {
        "workload": "configs[%d] %s" % (w.index, w.name),
        "value_ms": nums["train"] + nums["prefill"] + sum(t_dec), "ms_per_step": nums["total"],
        "phases_ms": {"train_fwd": nums["train"], "prefill": nums["prefill"], "decode": t_dec, "logprob": nums["logprob"]},
        "train_fwd": tensor(w.train_flops(), nums["train"], nums["alone_train"]),
        "prefill": tensor(w.prefill_flops(), nums["prefill"], nums["alone_prefill"]),
        "logprob": tensor(w.logprob_flops(), nums["logprob"]),
        "decode": [], "clocks": clk,
    }
    for i, (d, t) in enumerate(zip(info["dec"], t_dec)):
        g = d["bytes"] / (t * 1e-3) / 1e9
        ta = nums["alone_decode%d" % i]
        ga = d["bytes"] / (ta * 1e-3) / 1e9
        tg = nums.get("graph_decode%d" % i, -1.0)
        graph = ({"ms_per_step": tg, "gbs": d["bytes"] / (tg * 1e-3) / 1e9, "frac_hbm": d["bytes"] / (tg * 1e-3) / 1e9 / hbm,
                  "note": "CUDA graph of 20 identical steps (L2 flush + decode + combine each), the same graph of "
                          "flushes alone taken off"} if tg > 0 else {"ms_per_step": None, "note": d.get("graph_note")})
        out["decode"].append({"context": d["label"], "ms": t, "gbs": g, "frac_hbm": g / hbm,
                              "frac_nominal_hbm": g / NOMINAL["hbm_gbs"], "unique_kv_bytes": d["bytes"],
                              "logical_kv_bytes": d["logical_bytes"],
                              "gbs_logical": d["logical_bytes"] / (t * 1e-3) / 1e9,
                              "tok_per_s": w.S * world / (t * 1e-3),
                              "alone": {"ms": ta, "gbs": ga, "frac_hbm": ga / hbm,
                                        "gbs_logical": d["logical_bytes"] / (ta * 1e-3) / 1e9},
                              "graph20": graph})
    wb = w.vocab * w.hidden * 2
    t = nums["logprob_decode_shaped"]
    out["logprob_decode_shaped"] = {"rows": info["lp_rows"], "ms": t, "weight_bytes": wb, "gbs": wb / (t * 1e-3) / 1e9,
                                    "frac_hbm": wb / (t * 1e-3) / 1e9 / hbm}
    if "replay_total" in nums:
        out["rollout_replay"] = {"total_ms": nums["replay_total"], **info["replay"],
                                 "note": "prefill + every decode step for real (cache write, decode, combine per step; "
                                         "the batch shrinks as sequences finish); launch-bound on small batches"}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=None,
                    help="time only this workload (0..4); default: all five, configs[4] is the headline")
    ap.add_argument("--impl", default="tik", choices=["tik", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip end-to-end, replay and the operators beside the step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "tik" else args.warmup

    rank, local_rank, world = tdist.env_world()
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    rank, local_rank, world = tdist.init("nccl")
    from paper_2609_35140_b200 import binding as tik
    tik.load()
    peaks, peak_src = load_peaks()
    burst, sust = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]

    head_idx = HEADLINE if args.workload is None else args.workload
    others = [i for i in range(5) if i != head_idx] if args.workload is None else []
    per_config, flags = {}, 0
    side_steps = max(3, min(args.steps, 5))
    for i in others:
        w = synth.get_workload(i)
        hp, nums, info = measure_workload(tik, w, side_steps, 3, rank, local_rank, False,
                                          want_replay=(i in (0, 1, 2)) and not args.no_extras)
        flags |= tik.device_status()
        nums = tdist.max_over_ranks(nums, device="cuda")
        if rank == 0:
            rep = report_workload(w, nums, info, peaks, world)
            rep["steps"], rep["warmup"] = side_steps, 3
            rep["gpu_launches"] = info["launches_timed"]
            per_config["configs[%d]" % i] = rep
        del hp
        gc.collect()
        torch.cuda.empty_cache()

    # ---- the headline workload: exactly --warmup untimed and --steps timed steps
    w = synth.get_workload(head_idx)
    hp, nums, info = measure_workload(tik, w, args.steps, args.warmup, rank, local_rank, True,
                                      want_replay=(head_idx in (0, 1, 2)) and not args.no_extras)
    e2e = None
    if not args.no_extras:
        e2e_steps = max(2, min(args.steps, 4))
        e2e_ms, h2d, d2h, pinned = time_e2e(hp, e2e_steps, 2)
        nums["e2e"] = e2e_ms
        e2e = {"h2d": h2d, "d2h": d2h, "pinned": pinned, "steps": e2e_steps}
    flags |= tik.device_status()
    nums = tdist.max_over_ranks(nums, device="cuda")
    if rank != 0:
        tdist.finalize()
        return

    head = report_workload(w, nums, info, peaks, world)
    head["steps"], head["warmup"] = args.steps, args.warmup
    head["gpu_launches"] = info["launches_timed"]
    per_config["configs[%d]" % head_idx] = head
    clk = info["clocks"]
    # The headline's timed region runs for seconds with the log-prob GEMM drawing ~1 kW: when the
    # sampled median SM clock is below 90 % of the maximum AND the region lasted over a second, the
    # tensor-bound kernels are held against the sustained bf16 peak, otherwise against the burst peak.
    capped = bool(clk.get("sm_mhz")) and bool(clk.get("sm_max_mhz")) and clk["sm_mhz"] < 0.9 * clk["sm_max_mhz"]
    long_region = nums["total"] * args.steps >= 1000.0
    tpeak, tkind = (sust, "sustained") if (capped and long_region) else (burst, "burst")

    def tensor_roof(block, note=None):
        r = {"bound": "tensor", "achieved": block["tflops"], "peak": tpeak, "peak_kind": tkind, "unit": "TFLOP/s",
             "frac": block["tflops"] / tpeak, "frac_burst_peak": block["frac_burst_peak"],
             "frac_sustained_peak": block["frac_sustained_peak"], "frac_nominal_peak": block["frac_nominal_peak"],
             "ms": block["ms"]}
        if "alone" in block:
            r["alone_at_its_own_clocks"] = block["alone"]
        if note:
            r["note"] = note
        return r

    rooflines = {"train_fwd": tensor_roof(head["train_fwd"]),
                 "prefill": tensor_roof(head["prefill"], "includes the KV-cache write"),
                 "logprob": tensor_roof(head["logprob"])}
    for d in head["decode"]:
        rooflines["decode@%s" % d["context"]] = {
            "bound": "hbm", "achieved": d["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": d["frac_hbm"],
            "ms": d["ms"], "unique_kv_bytes": d["unique_kv_bytes"], "tok_per_s": d["tok_per_s"],
            "alone": d["alone"], "note": "attention + combine kernels"}
    ld = head["logprob_decode_shaped"]
    rooflines["logprob_decode_shaped"] = {"bound": "hbm", "achieved": ld["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                          "frac": ld["frac_hbm"], "ms": ld["ms"],
                                          "note": "T=%d rows (one per sequence): lm_head bytes V*H*2 over the launch time" % ld["rows"]}
    # the dominant kernel of `value` (the attention phases) by time
    dom_name = max(("train_fwd", "prefill"), key=lambda n: rooflines[n]["ms"])
    dom = rooflines[dom_name]
    traffic = None
    if NCU_TRAFFIC["bytes_per_token"] and dom_name == "train_fwd" and w.index == HEADLINE:
        traffic = NCU_TRAFFIC["bytes_per_token"] * w.total_tokens
    roofline = {"kernel": {"train_fwd": "attn_persist_kernel<128,packed>", "prefill": "attn_persist_kernel<128,paged>"}[dom_name],
                "bound": "tensor", "achieved": dom["achieved"], "peak": dom["peak"], "unit": "TFLOP/s",
                "frac": dom["frac"], "traffic": traffic, "traffic_source": NCU_TRAFFIC["source"],
                "peak_source": "of %s (%s bf16 peak: median SM clock %s of %s MHz over a timed region of %.1f s)" % (
                    peak_src, tkind, clk.get("sm_mhz"), clk.get("sm_max_mhz"), nums["total"] * args.steps / 1e3),
                "frac_burst_peak": dom["frac_burst_peak"], "frac_sustained_peak": dom["frac_sustained_peak"],
                "frac_nominal_peak": dom["frac_nominal_peak"],
                "algorithmic_flops_per_launch": w.train_flops() if dom_name == "train_fwd" else w.prefill_flops()}

    if world == 1 and not args.no_extras:
        t_prep, b_prep = time_prep(hp)
        g = b_prep / (t_prep * 1e-3) / 1e9
        rooflines["qk_norm_rope_kv_write"] = {
            "bound": "hbm", "achieved": g, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": g / peaks["hbm_gbs"],
            "ms": t_prep, "bytes": b_prep,
            "note": "pre-attention step over all tokens of the workload; measured after the timed steps, not part of the metric"}
        rooflines["attn_train_bwd"] = time_bwd(hp, burst)
        rooflines.update(time_ffn(hp, peaks, burst))    # timed alone: held against the burst peak
        flags |= tik.device_status()

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        ms, cores, desc, _ = oracle_sample_ms(w)
        cpu = {"value": ms, "unit": "ms", "cores": cores, "kind": "oracle", "sample": desc}

    side_launches = sum(per_config[k]["gpu_launches"] for k in per_config if k != "configs[%d]" % head_idx)
    line = {
        "metric": METRIC, "value": head["value_ms"], "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": nums["total"], "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, world),
        "phases_ms": head["phases_ms"],
        "decode_tok_per_s": [d["tok_per_s"] for d in head["decode"]],
        "roofline": roofline, "rooflines": rooflines, "cpu_baseline": cpu,
        "e2e": {"value": nums.get("e2e"), "unit": "ms",
                "h2d_bytes_per_step": e2e["h2d"] if e2e else 0, "d2h_bytes_per_step": e2e["d2h"] if e2e else 0,
                "steps": e2e["steps"] if e2e else 0, "pinned_host_bytes": e2e["pinned"] if e2e else 0,
                "note": "attention phases; every step stages its inputs from pageable host memory through a bounded ring of "
                        "pinned slots (one cudaMemcpyAsync per 128 MiB slice) and copies its outputs back through a second "
                        "ring; copies of neighbouring steps overlap the kernels (three streams, two device buffer sets)"},
        "per_config": per_config,
        "gpu_launches": info["launches_timed"],
        "gpu_launches_other_configs": side_launches,
        "clocks": clk, "device_flags": flags, "contract": tik.contract_id(),
    }
    print(json.dumps(line))
    tdist.finalize()


if __name__ == "__main__":
    main()
