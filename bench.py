#!/usr/bin/env python
"""Benchmark of the unified attention + token log-prob hot path on B200.

One step = one pass of the whole hot path over one synthetic workload:
  train-forward attention over all packed sequences
  -> KV-cache write + prefill attention over the prompts
  -> one decode step (attention + split-KV combine) per timed context
  -> token log-probabilities over all response tokens.
Headline metric: summed train-forward + prefill + decode attention time (ms, lower is
better); decode tokens/s, the log-prob time and per-kernel roofline fractions ride along.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--impl tik|reference]

N > 1 (torchrun, one rank per GPU): N independent replicas, no collective on the data path;
the reported times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
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

METRIC = "summed_attention_ms"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per launch of the dominant kernel from one ncu capture (profiles/), keyed by
# workload index; None until captured.
NCU_TRAFFIC_BYTES = {1: 3485940960}     # logprob_kernel on workload 1: 3.454 GB read + 32.2 MB written


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

    def result(self):
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
                "bytes": self._decode_bytes(lens), "label": c or "full"})
        need = max(tik.workspace_bytes(tik.OP_ATTN_DECODE, w.S, w.Hq, w.Hkv, w.d, d["max"]) for d in self.dec)
        self.dec_ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
        self.o = torch.empty_like(self.q)
        # log-prob over all response tokens
        self.hidden, self.W, self.target = synth.make_logprob_inputs(w, dev, seed_offset=seed_offset)
        self.lp = torch.empty(self.hidden.shape[0], dtype=torch.float32, device=dev)
        need = tik.workspace_bytes(tik.OP_TOKEN_LOGPROB, self.hidden.shape[0], H=w.hidden, V=w.vocab)
        self.lp_ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
        self.flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        self.launches_per_step = 1 + 2 + 2 * len(self.dec) + 2

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

    # -- the calls of one step; `mark(name)` records an event after each phase
    def step(self, mark, flush=True):
        tik, w = self.tik, self.w
        if flush:
            self.flush.zero_()
        mark("flush0")
        tik.tik_attn_train_fwd(self.q, self.k, self.v, self.cu, max(w.seq_lens), w.softmax_scale, o=self.o)
        mark("train")
        if flush:
            self.flush.zero_()
        mark("flush1")
        tik.tik_kv_cache_write(self.pre_k, self.pre_v, self.pre_cu, self.pre_ctx, self.kc, self.vc, self.pre_bt)
        tik.tik_attn_prefill(self.pre_q, self.pre_cu, self.pre_ctx, self.kc, self.vc, self.pre_bt, self.pre_max,
                             self.pre_max, w.softmax_scale, o=self.pre_o)
        mark("prefill")
        for i, d in enumerate(self.dec):
            if flush:
                self.flush.zero_()
            mark("flushd%d" % i)
            tik.tik_attn_decode(d["q"], d["ctx"], self.kc, self.vc, self.bt, d["max"], w.softmax_scale,
                                ws=self.dec_ws, o=d["o"])
            mark("decode%d" % i)
        if flush:
            self.flush.zero_()
        mark("flush2")
        tik.tik_token_logprob(self.hidden, self.W, self.target, ws=self.lp_ws, logprob=self.lp)
        mark("logprob")


def time_steps(hp: HotPath, steps: int, warmup: int):
    """Returns (per-phase mean ms, total ms per step) measured with CUDA events."""
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        hp.step(lambda name: None)
    torch.cuda.synchronize()
    tdist.barrier()
    torch.cuda.synchronize()
    names, events = [], []
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


def time_e2e(hp: HotPath, steps: int, warmup: int, max_pinned_bytes: int = 6 << 30):
    """Attention phases end to end through the public API: every step copies its inputs in from
    pinned host memory and its outputs back.  Three streams and two sets of device buffers, as a
    serving or training loop would run it: the copy-in of step s+1 and the copy-out of step s-1
    run under the kernels of step s (PCIe is full duplex), so a step costs the longest of the
    three, not their sum.  Timed from the first copy-in to the last copy-out."""
    tik, w = hp.tik, hp.w
    comp = torch.cuda.current_stream()
    planned = sum(getattr(hp, n).numel() * getattr(hp, n).element_size() for n in ("q", "k", "v", "pre_q", "pre_k", "pre_v"))
    planned += hp.o.numel() * 2 + hp.pre_o.numel() * 2
    if planned > max_pinned_bytes:
        return None, 0, 0       # would pin too much host memory on a shared box
    host_in = {n: getattr(hp, n).cpu().pin_memory() for n in ("q", "k", "v", "cu", "pre_q", "pre_k", "pre_v")}
    host_in.update({"dq%d" % i: d["q"].cpu().pin_memory() for i, d in enumerate(hp.dec)})
    dev_in = [{n: torch.empty_like(t, device="cuda") for n, t in host_in.items()} for _ in range(2)]
    dev_out = [{"o": torch.empty_like(hp.o), "pre_o": torch.empty_like(hp.pre_o),
                **{"do%d" % i: torch.empty_like(d["o"]) for i, d in enumerate(hp.dec)}} for _ in range(2)]
    host_out = {n: torch.empty(t.shape, dtype=t.dtype).pin_memory() for n, t in dev_out[0].items()}
    h2d = sum(t.numel() * t.element_size() for t in host_in.values())
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    in_done = [torch.cuda.Event() for _ in range(2)]
    comp_done = [torch.cuda.Event() for _ in range(2)]
    out_done = [torch.cuda.Event() for _ in range(2)]

    def run(n_steps, t0=None, t1=None):
        for s in range(n_steps):
            b = s & 1
            with torch.cuda.stream(s_in):
                if s == 0 and t0 is not None:
                    t0.record(s_in)
                if s >= 2:
                    s_in.wait_event(comp_done[b])            # step s-2 has consumed this input set
                for n, t in host_in.items():
                    dev_in[b][n].copy_(t, non_blocking=True)
                in_done[b].record(s_in)
            comp.wait_event(in_done[b])
            if s >= 2:
                comp.wait_event(out_done[b])                 # step s-2's outputs have left this output set
            di, do = dev_in[b], dev_out[b]
            tik.tik_attn_train_fwd(di["q"], di["k"], di["v"], di["cu"], max(w.seq_lens), w.softmax_scale, o=do["o"])
            tik.tik_kv_cache_write(di["pre_k"], di["pre_v"], hp.pre_cu, hp.pre_ctx, hp.kc, hp.vc, hp.pre_bt)
            tik.tik_attn_prefill(di["pre_q"], hp.pre_cu, hp.pre_ctx, hp.kc, hp.vc, hp.pre_bt, hp.pre_max,
                                 hp.pre_max, w.softmax_scale, o=do["pre_o"])
            for i, d in enumerate(hp.dec):
                tik.tik_attn_decode(di["dq%d" % i], d["ctx"], hp.kc, hp.vc, hp.bt, d["max"], w.softmax_scale,
                                    ws=hp.dec_ws, o=do["do%d" % i])
            comp_done[b].record(comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[b])
                for n, t in host_out.items():
                    t.copy_(do[n], non_blocking=True)
                out_done[b].record(s_out)
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
    return t0.elapsed_time(t1) / steps, h2d, d2h


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
    times = []
    for _ in range(reps + 2):
        hp.flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        tik.tik_qk_norm_rope_kv_write(q, k, hp.v, wq, wk, 1e-6, tab, hp.cu, ctx, kc, vc, hp.bt)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    times = sorted(times[2:])
    # per token: q and k read and written, v read, K and V cache rows written, one table row read
    byt = w.total_tokens * ((w.Hq + w.Hkv) * w.d * 2 * 2 + 3 * w.Hkv * w.d * 2 + w.d * 4)
    return times[len(times) // 2], byt


def time_bwd(hp: "HotPath", burst, reps: int = 3):
    """The policy-update backward of the train-forward phase (dQ, dK, dV), timed on its own."""
    tik, w = hp.tik, hp.w
    gen = torch.Generator(device="cuda").manual_seed(w.seed + 777)
    do = torch.randn(hp.q.shape, generator=gen, device="cuda").to(torch.bfloat16)
    lse = torch.empty(hp.q.shape[0], w.Hq, dtype=torch.float32, device="cuda")
    o = tik.tik_attn_train_fwd(hp.q, hp.k, hp.v, hp.cu, max(w.seq_lens), w.softmax_scale, lse=lse)
    ws = torch.empty(max(16, tik.workspace_bytes(tik.OP_ATTN_TRAIN_BWD, hp.q.shape[0], w.Hq, w.Hkv, w.d)),
                     dtype=torch.uint8, device="cuda")
    ts = []
    for _ in range(reps + 1):
        hp.flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        tik.tik_attn_train_bwd(hp.q, hp.k, hp.v, o, do, lse, hp.cu, max(w.seq_lens), w.softmax_scale, ws=ws)
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    ms = sorted(ts[1:])[len(ts[1:]) // 2]
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

    def med(fn):
        ts = []
        for _ in range(reps + 2):
            hp.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ts = sorted(ts[2:])
        return ts[len(ts) // 2]

    def hbm(ms, byt, note):
        g = byt / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": g, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": g / peaks["hbm_gbs"],
                "ms": ms, "bytes": byt, "note": note}

    def tensor(ms, flops, note):
        tf = flops / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak, "ms": ms,
                "note": note}

    shape = "T=%d H=%d I=%d; beside the step, not part of the metric" % (T, H, I)
    r = {}
    r["rmsnorm"] = hbm(med(lambda: tik.tik_rmsnorm(x, wn, 1e-6, y=h)), 2 * T * H * 2, shape)
    r["add_rmsnorm"] = hbm(med(lambda: tik.tik_rmsnorm(x, wn, 1e-6, residual=res, y=h)), 4 * T * H * 2, shape)
    r["linear_gate_up"] = tensor(med(lambda: tik.tik_linear(h, w_gu, y=gu)), 2.0 * T * H * 2 * I, shape)
    r["swiglu"] = hbm(med(lambda: tik.tik_swiglu(gu, out=act)), 3 * T * I * 2, shape)
    r["linear_down"] = tensor(med(lambda: tik.tik_linear(act, w_d, y=out)), 2.0 * T * I * H, shape)
    return r


# ------------------------------------------------------------------------------------------
def oracle_sample_ms(w: synth.Workload, budget_rows: int = 0, seed: int = 0):
    """Times the CPU oracle on a bounded sample of the workload's attention rows and scales
    by causal (query, key) pairs to the summed-attention metric.  Returns
    (extrapolated ms, cores, description, measured seconds)."""
    import oracle
    rng = np.random.default_rng(w.seed + 555 + seed)
    cu = w.cu_seqlens()
    G = w.G
    # metric pairs: train rows + prefill rows + decode rows (per query head)
    firsts = {}
    for s, g in enumerate(w.group_of):
        firsts.setdefault(g, s)
    pre_pairs = sum(w.prompt_lens[s] * (w.prompt_lens[s] + 1) // 2 for s in firsts.values())
    ctxs = w.decode_contexts or [None]
    dec_pairs = sum(sum(min(L, c) if c else L for L in w.seq_lens) for c in ctxs)
    metric_pairs = (w.causal_pairs() + pre_pairs + dec_pairs) * w.Hq
    # one KV head's K/V for every sequence, then random (sequence, position) rows until the
    # sample holds about 2.5e8 query-key pairs (10-20 s on 8 cores)
    target_pairs = 2.5e8
    gen = torch.Generator().manual_seed(w.seed + 99)
    rows, offs, lens = [], [], []
    kparts, vparts = [], []
    starts = []
    base = 0
    for s in range(w.S):
        L = w.seq_lens[s]
        kparts.append(torch.randn(L, w.d, generator=gen).to(torch.bfloat16).float().numpy())
        vparts.append(torch.randn(L, w.d, generator=gen).to(torch.bfloat16).float().numpy())
        starts.append(base)
        base += L
    pairs = 0
    while pairs < min(target_pairs, metric_pairs):
        s = int(rng.integers(0, w.S))
        t = int(rng.integers(0, w.seq_lens[s]))
        rows.append(1)
        offs.append(starts[s])
        lens.append(t + 1)
        pairs += t + 1
    kflat, vflat = np.concatenate(kparts), np.concatenate(vparts)
    qrows = torch.randn(len(rows), w.d, generator=gen).to(torch.bfloat16).float().numpy()
    t0 = time.perf_counter()
    oracle.attn_rows(qrows, kflat, vflat, offs, lens, w.softmax_scale)
    dt = time.perf_counter() - t0
    ms = dt * 1e3 * (metric_pairs / max(pairs, 1))
    desc = ("oracle.attn_rows on %d sampled rows (%.3g of %.3g causal query-key pairs of train+prefill+decode), "
            "%.2f s measured, scaled by pairs" % (len(rows), pairs, metric_pairs, dt))
    return ms, oracle.num_threads(), desc, dt


def run_reference(args, rank, world):
    if rank != 0:
        return
    w = synth.get_workload(args.workload)
    vals = []
    desc, cores = "", 0
    for i in range(args.warmup + args.steps):
        ms, cores, desc, _ = oracle_sample_ms(w, seed=i)
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
            "l2": "a 512 MiB buffer is overwritten before every phase (L2 flush), excluded from the phase times",
            "parallelism": "replicas x%d (no collective)" % n_gpus}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=1, help="index into the five workloads (default 1: 1.5B-class)")
    ap.add_argument("--impl", default="tik", choices=["tik", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
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

    w = synth.get_workload(args.workload)
    hp = HotPath(tik, w, seed_offset=tdist.replica_seed_offset(rank))
    torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    phase, total_ms = time_steps(hp, args.steps, args.warmup)
    sampler.stop_flag.set()
    sampler.join()
    e2e_ms, h2d, d2h = time_e2e(hp, max(4, args.steps), 2)
    flags = tik.device_status()

    local = dict(phase)
    local["total"] = total_ms
    local["e2e"] = e2e_ms if e2e_ms is not None else -1.0
    agg = tdist.max_over_ranks(local, device="cuda")
    if rank != 0:
        tdist.finalize()
        return

    peaks, peak_src = load_peaks()
    dec_keys = sorted(k for k in agg if k.startswith("decode"))
    t_train, t_prefill, t_lp = agg["train"], agg["prefill"], agg["logprob"]
    t_dec = [agg[k] for k in dec_keys]
    value = t_train + t_prefill + sum(t_dec)
    tf_train = w.train_flops() / (t_train * 1e-3) / 1e12
    tf_pre = w.prefill_flops() / (t_prefill * 1e-3) / 1e12
    tf_lp = w.logprob_flops() / (t_lp * 1e-3) / 1e12
    dec_gbs = [d["bytes"] / (t * 1e-3) / 1e9 for d, t in zip(hp.dec, t_dec)]
    burst, sust = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    # A kernel timed inside a long, power-capped step is held against the sustained tensor peak,
    # one that ran at (nearly) full clocks against the burst peak; both fractions are reported.
    clk = sampler.result()
    capped = bool(clk.get("sm_mhz")) and bool(clk.get("sm_max_mhz")) and clk["sm_mhz"] < 0.9 * clk["sm_max_mhz"]
    tpeak, tkind = (sust, "sustained") if capped else (burst, "burst")

    def tensor_roof(tf, ms, note=None):
        r = {"bound": "tensor", "achieved": tf, "peak": tpeak, "peak_kind": tkind, "unit": "TFLOP/s",
             "frac": tf / tpeak, "frac_burst_peak": tf / burst, "frac_sustained_peak": tf / sust, "ms": ms}
        if note:
            r["note"] = note
        return r

    rooflines = {
        "train_fwd": tensor_roof(tf_train, t_train),
        "prefill": tensor_roof(tf_pre, t_prefill, "includes the KV-cache write"),
        "logprob": tensor_roof(tf_lp, t_lp),
    }
    for d, t, g in zip(hp.dec, t_dec, dec_gbs):
        rooflines["decode@%s" % d["label"]] = {
            "bound": "hbm", "achieved": g, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": g / peaks["hbm_gbs"], "ms": t, "unique_kv_bytes": d["bytes"],
            "tok_per_s": w.S / (t * 1e-3), "note": "attention + combine kernels"}
    # the dominant kernel of the step by time
    dom_name = max(("train_fwd", "prefill", "logprob"), key=lambda n: rooflines[n]["ms"])
    dom = rooflines[dom_name]
    roofline = {"kernel": {"train_fwd": "attn_kernel<128,train>", "prefill": "attn_kernel<128,prefill>",
                           "logprob": "logprob_kernel<pair>"}[dom_name],
                "bound": dom["bound"], "achieved": dom["achieved"], "peak": dom["peak"], "unit": dom["unit"],
                "frac": dom["frac"], "traffic": NCU_TRAFFIC_BYTES.get(w.index),
                "peak_source": "of %s (%s bf16 peak: median SM clock %s of %s MHz in the timed region)" % (
                    peak_src, tkind, clk.get("sm_mhz"), clk.get("sm_max_mhz")),
                "frac_burst_peak": dom["frac_burst_peak"], "frac_sustained_peak": dom["frac_sustained_peak"]}

    if world == 1:
        t_prep, b_prep = time_prep(hp)
        g = b_prep / (t_prep * 1e-3) / 1e9
        rooflines["qk_norm_rope_kv_write"] = {
            "bound": "hbm", "achieved": g, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": g / peaks["hbm_gbs"],
            "ms": t_prep, "bytes": b_prep,
            "note": "pre-attention step over all tokens of the workload; measured after the timed steps, not part of the metric"}
        rooflines.update(time_ffn(hp, peaks, burst))    # timed alone: held against the burst peak
        rooflines["attn_train_bwd"] = time_bwd(hp, burst)
        flags |= tik.device_status()

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        ms, cores, desc, _ = oracle_sample_ms(w)
        cpu = {"value": ms, "unit": "ms", "cores": cores, "kind": "oracle", "sample": desc}

    line = {
        "metric": METRIC, "value": value, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": agg["total"], "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, world),
        "phases_ms": {"train_fwd": t_train, "prefill": t_prefill, "decode": t_dec, "logprob": t_lp},
        "decode_tok_per_s": [w.S * world / (t * 1e-3) for t in t_dec],
        "roofline": roofline, "rooflines": rooflines, "cpu_baseline": cpu,
        "e2e": {"value": agg["e2e"] if agg["e2e"] >= 0 else None, "unit": "ms", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "attention phases with pinned-host inputs copied in and outputs copied back each step; copies of neighbouring steps overlap the kernels (three streams, two buffer sets)"},
        "gpu_launches": hp.launches_per_step * args.steps,
        "clocks": clk, "device_flags": flags, "contract": tik.contract_id(),
    }
    print(json.dumps(line))
    tdist.finalize()


if __name__ == "__main__":
    main()
