"""ctypes binding of libtik.so: argument marshalling only.

Every function takes torch CUDA tensors (device memory and the current
stream come from torch), checks dtypes/contiguity, and forwards raw pointers
and sizes to the C entry point of the same name.  All arithmetic happens in
the library's kernels; there is no fallback, and a missing library raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

OK = 0
OP_ATTN_TRAIN_FWD, OP_ATTN_PREFILL, OP_ATTN_DECODE, OP_TOKEN_LOGPROB, OP_ATTN_TRAIN_BWD = 0, 1, 2, 3, 4
DEV_BAD_BLOCK, DEV_BAD_TARGET, DEV_WAIT_EXPIRED, DEV_BAD_POSITION, DEV_BAD_CONTEXT = 1, 2, 4, 8, 16

_lib = None
_ctx = {}


class TikError(RuntimeError):
    pass


def load(build_if_missing: bool = False) -> ctypes.CDLL:
    """Loads libtik.so (optionally building it first).  Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if build_if_missing:
        _build.build()
    if not os.path.exists(path):
        raise TikError("libtik.so is not built (%s); run `python -m paper_2609_35140_b200.build`. "
                       "There is no fallback path." % path)
    lib = ctypes.CDLL(path)
    c = ctypes
    vp, i32, i64, f32, sz = c.c_void_p, c.c_int, c.c_int64, c.c_float, c.c_size_t
    lib.tik_create.argtypes = [c.POINTER(vp), i32]
    lib.tik_destroy.argtypes = [vp]
    lib.tik_status_str.argtypes = [i32]
    lib.tik_status_str.restype = c.c_char_p
    lib.tik_last_error.argtypes = [vp]
    lib.tik_last_error.restype = c.c_char_p
    lib.tik_contract_id.restype = c.c_char_p
    lib.tik_kernel_launches.restype = c.c_ulonglong
    lib.tik_kernel_launches.argtypes = []
    lib.tik_workspace_bytes.argtypes = [i32, i64, i32, i32, i32, i64, i32, i32]
    lib.tik_workspace_bytes.restype = sz
    lib.tik_device_status.argtypes = [vp, vp, c.POINTER(i32)]
    lib.tik_attn_train_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32, vp, sz, vp]
    lib.tik_kv_cache_write.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i32, i32, i32, i32, vp]
    lib.tik_attn_prefill.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i32, i32, i32, i32,
                                     i32, i32, i32, f32, vp, sz, vp]
    lib.tik_attn_prefill_kv.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i32, i32, i32, i32,
                                        i32, i32, i32, f32, vp, sz, vp]
    lib.tik_attn_prefill_kv.restype = i32
    lib.tik_attn_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32,
                                    f32, vp, sz, vp]
    lib.tik_qk_norm_rope_kv_write.argtypes = [vp, vp, vp, vp, vp, vp, f32, vp, i32, vp, vp, vp, vp, vp, i32, i32,
                                              i64, i32, i32, i32, i32, i32, vp]
    lib.tik_rmsnorm.argtypes = [vp, vp, vp, vp, vp, f32, i64, i32, vp]
    lib.tik_swiglu.argtypes = [vp, vp, vp, i64, i32, vp]
    lib.tik_linear.argtypes = [vp, vp, vp, vp, i64, i32, i32, vp]
    lib.tik_attn_train_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, f32,
                                       vp, sz, vp]
    lib.tik_token_logprob.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, i32, f32, vp, sz, vp]
    lib.tik_attn_decode_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                           i32, f32, vp, vp]
    lib.tik_attn_decode_static.restype = i32
    for name in ("tik_create", "tik_destroy", "tik_device_status", "tik_attn_train_fwd",
                 "tik_kv_cache_write", "tik_attn_prefill", "tik_attn_decode", "tik_token_logprob",
                 "tik_qk_norm_rope_kv_write", "tik_rmsnorm", "tik_swiglu", "tik_linear",
                 "tik_attn_train_bwd"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def contract_id() -> str:
    return load().tik_contract_id().decode()


def context(device: Optional[int] = None) -> ctypes.c_void_p:
    """The per-device library context (created on first use)."""
    lib = load()
    if not torch.cuda.is_available():
        raise TikError("tik needs a CUDA device; there is no CPU path")
    dev = torch.cuda.current_device() if device is None else device
    if dev not in _ctx:
        h = ctypes.c_void_p()
        rc = lib.tik_create(ctypes.byref(h), dev)
        if rc != OK:
            raise TikError("tik_create failed: %s" % lib.tik_status_str(rc).decode())
        _ctx[dev] = h
    return _ctx[dev]


def _check(rc: int, ctx) -> None:
    if rc != OK:
        lib = load()
        raise TikError("%s: %s" % (lib.tik_status_str(rc).decode(), lib.tik_last_error(ctx).decode()))


def _ptr(t: Optional[torch.Tensor], dtype=None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise TikError("tensors must be contiguous CUDA tensors")
    if dtype is not None and t.dtype != dtype:
        raise TikError("expected dtype %s, got %s" % (dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def workspace_bytes(op: int, rows_or_batch: int = 0, Hq: int = 0, Hkv: int = 0, d: int = 0,
                    max_ctx: int = 0, H: int = 0, V: int = 0) -> int:
    return int(load().tik_workspace_bytes(op, rows_or_batch, Hq, Hkv, d, max_ctx, H, V))


def kernel_launches() -> int:
    """Kernels the library has launched in this process so far."""
    return int(load().tik_kernel_launches())


def device_status() -> int:
    """Synchronises the current stream; returns and clears the device flags."""
    ctx = context()
    flags = ctypes.c_int(0)
    _check(load().tik_device_status(ctx, _stream(), ctypes.byref(flags)), ctx)
    return flags.value


def _plan_ws(op: int, S: int, max_positions: int, ws, device):
    """Scratch of the full-sequence kernels: None -> allocate what the op asks for (persistent
    schedule), False -> pass none (one CTA per work item), a tensor -> use it."""
    if ws is False:
        return None
    if ws is None:
        need = workspace_bytes(op, S, max_ctx=max_positions)
        return torch.empty(need, dtype=torch.uint8, device=device) if need > 0 else None
    return ws


def tik_attn_train_fwd(q, k, v, cu_seqlens, max_seqlen: int, softmax_scale: float,
                       o: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None, ws=None):
    """q [tot,Hq,d], k/v [tot,Hkv,d] bf16, cu_seqlens int32 [S+1] (device) -> o [tot,Hq,d].
    ws: scratch tensor, None (allocated here) or False (run without: one CTA per work item)."""
    ctx = context()
    tot, Hq, d = q.shape
    Hkv = k.shape[1]
    if o is None:
        o = torch.empty_like(q)
    bf = torch.bfloat16
    ws = _plan_ws(OP_ATTN_TRAIN_FWD, cu_seqlens.numel() - 1, max_seqlen, ws, q.device)
    rc = load().tik_attn_train_fwd(ctx, _ptr(q, bf), _ptr(k, bf), _ptr(v, bf), _ptr(o, bf),
                                   _ptr(lse, torch.float32), _ptr(cu_seqlens, torch.int32),
                                   cu_seqlens.numel() - 1, tot, max_seqlen, Hq, Hkv, d,
                                   softmax_scale, _ptr(ws), ws.numel() if ws is not None else 0, _stream())
    _check(rc, ctx)
    return o


def tik_attn_train_bwd(q, k, v, o, d_o, lse, cu_seqlens, max_seqlen: int, softmax_scale: float,
                       ws: Optional[torch.Tensor] = None):
    """Backward of tik_attn_train_fwd: returns (dq, dk, dv).  o, lse are the forward's outputs."""
    ctx = context()
    bf = torch.bfloat16
    tot, Hq, d = q.shape
    Hkv = k.shape[1]
    need = workspace_bytes(OP_ATTN_TRAIN_BWD, tot, Hq, Hkv, d)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    rc = load().tik_attn_train_bwd(ctx, _ptr(q, bf), _ptr(k, bf), _ptr(v, bf), _ptr(o, bf), _ptr(d_o, bf),
                                   _ptr(lse, torch.float32), _ptr(dq, bf), _ptr(dk, bf), _ptr(dv, bf),
                                   _ptr(cu_seqlens, torch.int32), cu_seqlens.numel() - 1, tot, max_seqlen, Hq, Hkv, d,
                                   softmax_scale, _ptr(ws), ws.numel(), _stream())
    _check(rc, ctx)
    return dq, dk, dv


def tik_kv_cache_write(k_new, v_new, cu_seqlens_new, ctx_lens, k_cache, v_cache, block_table):
    """Copies new K/V rows into the paged caches [num_pages,Hkv,page,d] in place."""
    ctx = context()
    bf = torch.bfloat16
    num_pages, Hkv, page, d = k_cache.shape
    rc = load().tik_kv_cache_write(ctx, _ptr(k_new, bf), _ptr(v_new, bf),
                                   _ptr(cu_seqlens_new, torch.int32), _ptr(ctx_lens, torch.int32),
                                   _ptr(k_cache, bf), _ptr(v_cache, bf),
                                   _ptr(block_table, torch.int32), block_table.shape[1],
                                   ctx_lens.numel(), k_new.shape[0], Hkv, d, page, num_pages, _stream())
    _check(rc, ctx)


def tik_qk_norm_rope_kv_write(q, k, v, q_weight, k_weight, eps: float, cos_sin, cu_seqlens_new,
                              ctx_lens=None, k_cache=None, v_cache=None, block_table=None):
    """Per-head RMSNorm (weights may be None) and NeoX RoPE of q [n,Hq,d] and k [n,Hkv,d] in place;
    with caches, rotated K and V also go to the pages.  cos_sin fp32 [max_pos,d]."""
    ctx = context()
    bf = torch.bfloat16
    n, Hq, d = q.shape
    Hkv = k.shape[1]
    page = k_cache.shape[2] if k_cache is not None else 0
    num_pages = k_cache.shape[0] if k_cache is not None else 0
    rc = load().tik_qk_norm_rope_kv_write(
        ctx, _ptr(q, bf), _ptr(k, bf), _ptr(v, bf), _ptr(q_weight, bf), _ptr(k_weight, bf), float(eps),
        _ptr(cos_sin, torch.float32), cos_sin.shape[0], _ptr(cu_seqlens_new, torch.int32),
        _ptr(ctx_lens, torch.int32), _ptr(k_cache, bf), _ptr(v_cache, bf), _ptr(block_table, torch.int32),
        block_table.shape[1] if block_table is not None else 0, cu_seqlens_new.numel() - 1, n, Hq, Hkv, d,
        page, num_pages, _stream())
    _check(rc, ctx)


def tik_rmsnorm(x, weight, eps: float, residual=None, y: Optional[torch.Tensor] = None):
    """RMSNorm of x [T,H] over H; with residual [T,H], residual <- bf16(x + residual) first and that
    sum is normalised.  Returns y [T,H]."""
    ctx = context()
    bf = torch.bfloat16
    T, H = x.shape
    if y is None:
        y = torch.empty_like(x)
    rc = load().tik_rmsnorm(ctx, _ptr(x, bf), _ptr(residual, bf), _ptr(weight, bf), _ptr(y, bf), float(eps),
                            T, H, _stream())
    _check(rc, ctx)
    return y


def tik_swiglu(gate_up, out: Optional[torch.Tensor] = None):
    """gate_up [T,2I] (gate | up) -> silu(gate) * up, [T,I]."""
    ctx = context()
    bf = torch.bfloat16
    T, I2 = gate_up.shape
    if out is None:
        out = torch.empty(T, I2 // 2, dtype=bf, device=gate_up.device)
    rc = load().tik_swiglu(ctx, _ptr(gate_up, bf), _ptr(out, bf), T, I2 // 2, _stream())
    _check(rc, ctx)
    return out


def tik_linear(x, weight, y: Optional[torch.Tensor] = None):
    """x [T,K] @ weight[N,K]^T -> y [T,N] (bf16, fp32 accumulation)."""
    ctx = context()
    bf = torch.bfloat16
    T, K = x.shape
    N = weight.shape[0]
    if y is None:
        y = torch.empty(T, N, dtype=bf, device=x.device)
    rc = load().tik_linear(ctx, _ptr(x, bf), _ptr(weight, bf), _ptr(y, bf), T, K, N, _stream())
    _check(rc, ctx)
    return y


def tik_attn_prefill(q, cu_seqlens_q, ctx_lens, k_cache, v_cache, block_table, max_q_len: int,
                     max_ctx_len: int, softmax_scale: float, o: Optional[torch.Tensor] = None,
                     lse: Optional[torch.Tensor] = None, ws=None):
    """q [totq,Hq,d] against the paged cache -> o [totq,Hq,d].  ws as for tik_attn_train_fwd."""
    ctx = context()
    bf = torch.bfloat16
    totq, Hq, d = q.shape
    num_pages, Hkv, page, _ = k_cache.shape
    if o is None:
        o = torch.empty_like(q)
    ws = _plan_ws(OP_ATTN_PREFILL, ctx_lens.numel(), max_ctx_len, ws, q.device)
    rc = load().tik_attn_prefill(ctx, _ptr(q, bf), _ptr(o, bf), _ptr(lse, torch.float32),
                                 _ptr(cu_seqlens_q, torch.int32), _ptr(ctx_lens, torch.int32),
                                 _ptr(k_cache, bf), _ptr(v_cache, bf), _ptr(block_table, torch.int32),
                                 block_table.shape[1], ctx_lens.numel(), totq, max_q_len, max_ctx_len,
                                 Hq, Hkv, d, page, num_pages, softmax_scale, _ptr(ws),
                                 ws.numel() if ws is not None else 0, _stream())
    _check(rc, ctx)
    return o


def tik_attn_prefill_kv(q, k_new, v_new, cu_seqlens_q, ctx_lens, k_cache, v_cache, block_table, max_q_len: int,
                        max_ctx_len: int, softmax_scale: float, o: Optional[torch.Tensor] = None,
                        lse: Optional[torch.Tensor] = None, ws=None):
    """Cache write of k_new / v_new [totq,Hkv,d] and prefill of q [totq,Hq,d] in one call -> o."""
    ctx = context()
    bf = torch.bfloat16
    totq, Hq, d = q.shape
    num_pages, Hkv, page, _ = k_cache.shape
    if o is None:
        o = torch.empty_like(q)
    ws = _plan_ws(OP_ATTN_PREFILL, ctx_lens.numel(), max_ctx_len, ws, q.device)
    rc = load().tik_attn_prefill_kv(ctx, _ptr(q, bf), _ptr(k_new, bf), _ptr(v_new, bf), _ptr(o, bf),
                                    _ptr(lse, torch.float32), _ptr(cu_seqlens_q, torch.int32),
                                    _ptr(ctx_lens, torch.int32), _ptr(k_cache, bf), _ptr(v_cache, bf),
                                    _ptr(block_table, torch.int32), block_table.shape[1], ctx_lens.numel(), totq,
                                    max_q_len, max_ctx_len, Hq, Hkv, d, page, num_pages, softmax_scale, _ptr(ws),
                                    ws.numel() if ws is not None else 0, _stream())
    _check(rc, ctx)
    return o


def tik_attn_decode(q, ctx_lens, k_cache, v_cache, block_table, max_ctx_len: int, softmax_scale: float,
                    ws: Optional[torch.Tensor] = None, o: Optional[torch.Tensor] = None,
                    lse: Optional[torch.Tensor] = None):
    """q [B,Hq,d]: one token per sequence against the paged cache -> o [B,Hq,d]."""
    ctx = context()
    bf = torch.bfloat16
    B, Hq, d = q.shape
    num_pages, Hkv, page, _ = k_cache.shape
    need = workspace_bytes(OP_ATTN_DECODE, B, Hq, Hkv, d, max_ctx_len)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    if o is None:
        o = torch.empty_like(q)
    rc = load().tik_attn_decode(ctx, _ptr(q, bf), _ptr(o, bf), _ptr(lse, torch.float32),
                                _ptr(ctx_lens, torch.int32), _ptr(k_cache, bf), _ptr(v_cache, bf),
                                _ptr(block_table, torch.int32), block_table.shape[1], B, max_ctx_len,
                                Hq, Hkv, d, page, num_pages, softmax_scale, _ptr(ws),
                                ws.numel() * ws.element_size(), _stream())
    _check(rc, ctx)
    return o


def tik_token_logprob(hidden, lm_head, target_ids, inv_temperature: float = 1.0,
                      ws: Optional[torch.Tensor] = None, logprob: Optional[torch.Tensor] = None,
                      lse: Optional[torch.Tensor] = None):
    """hidden [T,H], lm_head [V,H] bf16, target_ids int32 [T] -> logprob fp32 [T]."""
    ctx = context()
    bf = torch.bfloat16
    T, H = hidden.shape
    V = lm_head.shape[0]
    need = workspace_bytes(OP_TOKEN_LOGPROB, T, H=H, V=V)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=hidden.device)
    if logprob is None:
        logprob = torch.empty(T, dtype=torch.float32, device=hidden.device)
    rc = load().tik_token_logprob(ctx, _ptr(hidden, bf), _ptr(lm_head, bf), _ptr(target_ids, torch.int32),
                                  _ptr(logprob, torch.float32), _ptr(lse, torch.float32), T, H, V,
                                  inv_temperature, _ptr(ws), ws.numel() * ws.element_size(), _stream())
    _check(rc, ctx)
    return logprob


STATIC_SCRATCH_BYTES = 8 << 20


def tik_attn_decode_static(q, ctx_lens, k_cache, v_cache, block_table, max_ctx_len: int,
                           softmax_scale: float, o: torch.Tensor, lse: Optional[torch.Tensor] = None,
                           dev_flags: Optional[torch.Tensor] = None) -> int:
    """Decode attention through the entry point that allocates nothing: no library context,
    no workspace (the scratch is a fixed array inside the library) and, unlike the other
    wrappers, no output tensor is created here either - the caller passes `o`.  For callers
    whose device memory is fully committed or who cannot afford cudaMalloc's synchronisation.
    Returns the raw status code (0 = ok; -3 = the problem exceeds the fixed scratch)."""
    bf = torch.bfloat16
    B, Hq, d = q.shape
    num_pages, Hkv, page, _ = k_cache.shape
    return int(load().tik_attn_decode_static(
        _ptr(q, bf), _ptr(o, bf), _ptr(lse, torch.float32), _ptr(ctx_lens, torch.int32),
        _ptr(k_cache, bf), _ptr(v_cache, bf), _ptr(block_table, torch.int32), block_table.shape[1],
        B, max_ctx_len, Hq, Hkv, d, page, num_pages, softmax_scale, _ptr(dev_flags, torch.int32),
        _stream()))
