"""Single-kernel timings of the library on chosen shapes (also the command line for profiler captures).

Each case builds seeded synthetic inputs on the GPU, runs one entry point `--warmup` + `--reps`
times with an L2 flush before every launch (512 MiB written, then 256 MiB read; outside the timed span),
times every launch with CUDA events on the launching stream and prints one JSON line with the
median and minimum, the algorithmic work and the resulting rate.

  python -m paper_2609_35140_b200.microbench train   --seqs 1 --len 16384 --hq 32 --hkv 8
  python -m paper_2609_35140_b200.microbench prefill --seqs 32 --len 1024 --hq 64 --hkv 8
  python -m paper_2609_35140_b200.microbench decode  --seqs 16 --len 16384 --hq 32 --hkv 8
  python -m paper_2609_35140_b200.microbench logprob --rows 64 --hidden 3584 --vocab 152064
  python -m paper_2609_35140_b200.microbench linear  --rows 64 --hidden 3584 --out 18944
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as tik
from . import synth


class L2Flush:
    """Cold, clean L2 before a timed launch: a 512 MiB buffer is overwritten (nothing of the timed
    kernel's inputs survives in the 126 MB L2), then a 256 MiB buffer is read, which pushes the
    first pass's dirty lines out to HBM.  Without the read pass the timed kernel pays for writing
    back up to an L2-ful of the flush's own data (~15 us of HBM time on a B200)."""

    def __init__(self, device="cuda", read_pass: bool = True):
        self.w = torch.empty(512 << 20, dtype=torch.uint8, device=device)
        self.r = torch.zeros(64 << 20, dtype=torch.int32, device=device) if read_pass else None

    def zero_(self):            # same call as the plain buffer it replaces
        self.w.zero_()
        if self.r is not None:
            torch.sum(self.r)


def _time(fn, reps: int, warmup: int, flush):
    """Median and minimum launch time in ms.  All repetitions are queued before the one
    synchronisation, so the host's share of a call (tensor-map encoding, launch) overlaps the
    previous repetition's L2 flush as it would overlap the previous kernel in a real loop."""
    evs = []
    for i in range(warmup + reps):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    ts = sorted(e0.elapsed_time(e1) for e0, e1 in evs[warmup:])
    return ts[len(ts) // 2], ts[0]


def _lens(a):
    if a.workload >= 0:          # the first --first sequences of a benchmark workload (its length mix)
        w = synth.get_workload(a.workload)
        return w.seq_lens[:a.first] if a.first > 0 else w.seq_lens
    if a.lens:
        return [int(x) for x in a.lens.split(",")]
    return [a.len] * a.seqs


def paged_inputs(lens, Hq, Hkv, d, page, seed=1234, dev="cuda"):
    """Random caches with a shuffled block table covering `lens` keys per sequence."""
    gen = torch.Generator(device=dev).manual_seed(seed)
    nblk = [(L + page - 1) // page for L in lens]
    num_pages = sum(nblk) + 3
    perm = np.random.default_rng(seed).permutation(num_pages)
    bt = -np.ones((len(lens), max(nblk)), dtype=np.int32)
    nxt = 0
    for s, n in enumerate(nblk):
        bt[s, :n] = perm[nxt:nxt + n]
        nxt += n
    kc = synth._randn_bf16((num_pages, Hkv, page, d), gen, dev, chunk_rows=4096)
    vc = synth._randn_bf16((num_pages, Hkv, page, d), gen, dev, chunk_rows=4096)
    return kc, vc, torch.from_numpy(bt).to(dev), gen


def run(a) -> dict:
    tik.load()
    dev = "cuda"
    flush = None if a.no_flush else L2Flush(dev, read_pass=not a.write_only_flush)
    scale = float(np.float32(1.0 / np.sqrt(a.d)))
    out = {"case": a.case, "flush": not a.no_flush}
    if a.case == "train":
        lens = _lens(a)
        w = synth.custom_workload([1] * len(lens), [L - 1 for L in lens], a.hq, a.hkv, a.d, a.page)
        q, k, v, cu = synth.make_qkv(w, dev)
        o = torch.empty_like(q)
        wsarg = False if a.per_item else None
        med, mn = _time(lambda: tik.tik_attn_train_fwd(q, k, v, cu, max(lens), scale, o=o, ws=wsarg), a.reps, a.warmup, flush)
        fl = w.train_flops()
        out.update(shape={"lens": lens if len(lens) <= 8 else "%d x ..." % len(lens), "Hq": a.hq, "Hkv": a.hkv, "d": a.d},
                   flops=fl, tflops=fl / (med * 1e-3) / 1e12, tflops_best=fl / (mn * 1e-3) / 1e12)
    elif a.case == "prefill":
        lens = _lens(a)
        kc, vc, bt, gen = paged_inputs(lens, a.hq, a.hkv, a.d, a.page)
        q = synth._randn_bf16((sum(lens), a.hq, a.d), gen, dev)
        o = torch.empty_like(q)
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=dev)
        ctx = torch.tensor(lens, dtype=torch.int32, device=dev)
        wsarg = False if a.per_item else None
        med, mn = _time(lambda: tik.tik_attn_prefill(q, cu, ctx, kc, vc, bt, max(lens), max(lens), scale, o=o, ws=wsarg),
                        a.reps, a.warmup, flush)
        fl = 4.0 * a.d * a.hq * sum(L * (L + 1) // 2 for L in lens)
        out.update(shape={"prompts": len(lens), "len": max(lens), "Hq": a.hq, "Hkv": a.hkv, "d": a.d, "page": a.page},
                   flops=fl, tflops=fl / (med * 1e-3) / 1e12, tflops_best=fl / (mn * 1e-3) / 1e12)
    elif a.case == "decode":
        lens = _lens(a)
        kc, vc, bt, gen = paged_inputs(lens, a.hq, a.hkv, a.d, a.page)
        q = synth._randn_bf16((len(lens), a.hq, a.d), gen, dev)
        o = torch.empty_like(q)
        ctx = torch.tensor(lens, dtype=torch.int32, device=dev)
        ws = torch.empty(tik.workspace_bytes(tik.OP_ATTN_DECODE, len(lens), a.hq, a.hkv, a.d, max(lens)),
                         dtype=torch.uint8, device=dev)
        med, mn = _time(lambda: tik.tik_attn_decode(q, ctx, kc, vc, bt, max(lens), scale, ws=ws, o=o),
                        a.reps, a.warmup, flush)
        byt = sum(lens) * a.hkv * a.d * 2 * 2
        out.update(shape={"batch": len(lens), "ctx": max(lens), "Hq": a.hq, "Hkv": a.hkv, "d": a.d, "page": a.page},
                   kv_bytes=byt, gbs=byt / (med * 1e-3) / 1e9, gbs_best=byt / (mn * 1e-3) / 1e9)
    elif a.case in ("logprob", "linear"):
        gen = torch.Generator(device=dev).manual_seed(4321)
        n_out = a.vocab if a.case == "logprob" else a.out
        x = synth._randn_bf16((a.rows, a.hidden), gen, dev)
        W = synth._randn_bf16((n_out, a.hidden), gen, dev, std=0.02, chunk_rows=1 << 14)
        if a.case == "logprob":
            tgt = torch.randint(0, n_out, (a.rows,), generator=gen, device=dev, dtype=torch.int64).to(torch.int32)
            lp = torch.empty(a.rows, dtype=torch.float32, device=dev)
            ws = torch.empty(max(16, tik.workspace_bytes(tik.OP_TOKEN_LOGPROB, a.rows, H=a.hidden, V=n_out)),
                             dtype=torch.uint8, device=dev)
            fn = lambda: tik.tik_token_logprob(x, W, tgt, ws=ws, logprob=lp)
        else:
            y = torch.empty(a.rows, n_out, dtype=torch.bfloat16, device=dev)
            fn = lambda: tik.tik_linear(x, W, y=y)
        med, mn = _time(fn, a.reps, a.warmup, flush)
        fl = 2.0 * a.rows * a.hidden * n_out
        byt = n_out * a.hidden * 2
        out.update(shape={"rows": a.rows, "hidden": a.hidden, "out": n_out}, flops=fl, weight_bytes=byt,
                   tflops=fl / (med * 1e-3) / 1e12, weight_gbs=byt / (med * 1e-3) / 1e9,
                   weight_gbs_best=byt / (mn * 1e-3) / 1e9)
    else:
        raise SystemExit("unknown case " + a.case)
    out.update(ms=med, ms_best=mn, reps=a.reps, device_flags=tik.device_status())
    return out


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("case", choices=["train", "prefill", "decode", "logprob", "linear"])
    ap.add_argument("--seqs", type=int, default=1)
    ap.add_argument("--len", type=int, default=4096)
    ap.add_argument("--lens", default="", help="comma-separated lengths (overrides --seqs/--len)")
    ap.add_argument("--workload", type=int, default=-1, help="take the lengths of benchmark workload 0..4 (train / prefill / decode)")
    ap.add_argument("--first", type=int, default=0, help="with --workload: only its first N sequences")
    ap.add_argument("--hq", type=int, default=32)
    ap.add_argument("--hkv", type=int, default=8)
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--page", type=int, default=64)
    ap.add_argument("--rows", type=int, default=64)
    ap.add_argument("--hidden", type=int, default=4096)
    ap.add_argument("--vocab", type=int, default=151936)
    ap.add_argument("--out", type=int, default=12288)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--per-item", action="store_true", help="train / prefill without scratch: one CTA per work item")
    ap.add_argument("--write-only-flush", action="store_true", help="L2 flush without the read pass (dirty L2)")
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("microbench needs a CUDA device: the library has no CPU path")
    print(json.dumps(run(a)))


if __name__ == "__main__":
    main()
