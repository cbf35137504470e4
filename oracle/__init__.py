"""CPU oracle (test infrastructure only).

Thin numpy/ctypes wrapper over ``oracle.c``: plain, slow, one-row-at-a-time
definitions of causal grouped-query attention (Sec. 3.2 of the paper) and of
the token log-probability (Sec. 3.1).  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; it imports nothing
from the CUDA package and the CUDA package never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (OpenMP) into liboracle.so next to it."""
    srcs = [os.path.join(_HERE, "oracle.c"), os.path.join(_HERE, "oracle_impl.inc")]
    if not force and os.path.exists(_LIB_PATH):
        if all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in srcs):
            return _LIB_PATH
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", srcs[0], "-o", _LIB_PATH, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _real(f32: bool):
    return (np.float32, "_f32") if f32 else (np.float64, "")


def attn_packed(q, k, v, cu_seqlens, scale: float, f32: bool = False):
    """q [tot,Hq,d], k/v [tot,Hkv,d] -> (out [tot,Hq,d], lse [tot,Hq])."""
    q, k, v, cu = _f32(q), _f32(k), _f32(v), _i32(cu_seqlens)
    tot, Hq, d = q.shape
    Hkv = k.shape[1]
    assert k.shape == (tot, Hkv, d) and v.shape == k.shape and cu[-1] == tot
    dt, sfx = _real(f32)
    out = np.empty((tot, Hq, d), dtype=dt)
    lse = np.empty((tot, Hq), dtype=dt)
    rc = getattr(lib(), "oracle_attn_packed" + sfx)(
        _p(q), _p(k), _p(v), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(Hq),
        ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_double(scale), _p(out), _p(lse))
    assert rc == 0
    return out, lse


def attn_paged(q, cu_seqlens_q, ctx_lens, k_cache, v_cache, block_table, scale: float,
               f32: bool = False):
    """q [totq,Hq,d]; caches [num_pages,Hkv,page,d]; block_table [S,max_blocks]."""
    q, kc, vc = _f32(q), _f32(k_cache), _f32(v_cache)
    cu, ctx, bt = _i32(cu_seqlens_q), _i32(ctx_lens), _i32(block_table)
    totq, Hq, d = q.shape
    _, Hkv, page, d2 = kc.shape
    assert d2 == d and vc.shape == kc.shape and bt.ndim == 2 and bt.shape[0] == len(ctx)
    dt, sfx = _real(f32)
    out = np.empty((totq, Hq, d), dtype=dt)
    lse = np.empty((totq, Hq), dtype=dt)
    rc = getattr(lib(), "oracle_attn_paged" + sfx)(
        _p(q), _p(cu), _p(ctx), _p(kc), _p(vc), _p(bt), ctypes.c_int(bt.shape[1]),
        ctypes.c_int(len(ctx)), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d),
        ctypes.c_int(page), ctypes.c_double(scale), _p(out), _p(lse))
    assert rc == 0
    return out, lse


def attn_rows(q_rows, k, v, kv_off, kv_len, scale: float, f32: bool = False):
    """Row r: query q_rows[r] against k/v[kv_off[r] : kv_off[r]+kv_len[r]] (flat [totk,d])."""
    q_rows, k, v = _f32(q_rows), _f32(k), _f32(v)
    off, ln = _i64(kv_off), _i64(kv_len)
    n, d = q_rows.shape
    assert k.shape[1] == d and v.shape == k.shape
    assert n == 0 or int((off + ln).max()) <= k.shape[0]
    dt, sfx = _real(f32)
    out = np.empty((n, d), dtype=dt)
    lse = np.empty((n,), dtype=dt)
    rc = getattr(lib(), "oracle_attn_rows" + sfx)(
        _p(q_rows), _p(k), _p(v), _p(off), _p(ln), ctypes.c_int64(n), ctypes.c_int(d),
        ctypes.c_double(scale), _p(out), _p(lse))
    assert rc == 0
    return out, lse


def attn_probs(q_row, k, v, scale: float, f32: bool = False):
    """Normalised attention weights and output of one row over all rows of k/v [n,d]."""
    q_row, k, v = _f32(q_row), _f32(k), _f32(v)
    n, d = k.shape
    dt, sfx = _real(f32)
    probs = np.empty((n,), dtype=dt)
    out = np.empty((d,), dtype=dt)
    rc = getattr(lib(), "oracle_attn_probs" + sfx)(
        _p(q_row), _p(k), _p(v), ctypes.c_int64(n), ctypes.c_int(d), ctypes.c_double(scale),
        _p(probs), _p(out))
    assert rc == 0
    return probs, out


def token_logprob(hidden, W, target, inv_temperature: float = 1.0, f32: bool = False):
    """hidden [T,H], W [V,H], target [T] -> (logprob [T], lse [T])."""
    hidden, W, target = _f32(hidden), _f32(W), _i32(target)
    T, H = hidden.shape
    V = W.shape[0]
    assert W.shape[1] == H and target.shape == (T,)
    dt, sfx = _real(f32)
    lp = np.empty((T,), dtype=dt)
    lse = np.empty((T,), dtype=dt)
    rc = getattr(lib(), "oracle_token_logprob" + sfx)(
        _p(hidden), _p(W), _p(target), ctypes.c_int64(T), ctypes.c_int(H), ctypes.c_int(V),
        ctypes.c_double(inv_temperature), _p(lp), _p(lse))
    assert rc == 0
    return lp, lse


def log_softmax_row(hidden_row, W, inv_temperature: float = 1.0, f32: bool = False):
    """The full log-softmax row [V] of one token."""
    hidden_row, W = _f32(hidden_row), _f32(W)
    V, H = W.shape
    dt, sfx = _real(f32)
    out = np.empty((V,), dtype=dt)
    rc = getattr(lib(), "oracle_log_softmax_row" + sfx)(
        _p(hidden_row), _p(W), ctypes.c_int(H), ctypes.c_int(V),
        ctypes.c_double(inv_temperature), _p(out))
    assert rc == 0
    return out


def norm_rope(x, w, eps: float, cos_sin, pos, f32: bool = False):
    """x [T,H,d], w [d] or None, cos_sin [max_pos,d] (cos | sin), pos [T] -> RMSNorm then NeoX RoPE, [T,H,d]."""
    x, cos_sin, pos = _f32(x), _f32(cos_sin), _i64(pos)
    T, H, d = x.shape
    assert d % 2 == 0 and cos_sin.shape[1] == d and pos.shape == (T,)
    wp = None
    if w is not None:
        w = _f32(w)
        assert w.shape == (d,)
        wp = _p(w)
    dt, sfx = _real(f32)
    out = np.empty((T, H, d), dtype=dt)
    rc = getattr(lib(), "oracle_norm_rope" + sfx)(
        _p(x), wp, ctypes.c_double(eps), _p(cos_sin), ctypes.c_int64(cos_sin.shape[0]), _p(pos),
        ctypes.c_int64(T), ctypes.c_int(H), ctypes.c_int(d), _p(out))
    assert rc == 0, "position outside the cos/sin table"
    return out


def paged_scatter(rows, pos, block_table_row, page_size: int, cache):
    """Indexed KV-cache write as its plain definition: token i of one sequence, at position pos[i],
    goes to cache[block_table_row[pos[i] // page_size], :, pos[i] % page_size, :].  rows [n,Hkv,d];
    cache [num_pages,Hkv,page_size,d] is modified in place and returned."""
    for i, p in enumerate(pos):
        cache[int(block_table_row[int(p) // page_size]), :, int(p) % page_size, :] = rows[i]
    return cache


def rmsnorm(x, w, eps: float, residual=None, f32: bool = False):
    """x [T,H], w [H] -> y [T,H].  With residual [T,H]: s = bf16(x + residual) is normalised and
    also returned: (y, s)."""
    x, w = _f32(x), _f32(w)
    T, H = x.shape
    assert w.shape == (H,)
    res = None if residual is None else _f32(residual)
    dt, sfx = _real(f32)
    y = np.empty((T, H), dtype=dt)
    s = np.empty((T, H), dtype=np.float32) if res is not None else None
    rc = getattr(lib(), "oracle_rmsnorm" + sfx)(_p(x), _p(res), _p(w), ctypes.c_double(eps), ctypes.c_int64(T),
                                               ctypes.c_int(H), _p(y), _p(s))
    assert rc == 0
    return y if res is None else (y, s)


def swiglu(gate_up, f32: bool = False):
    """gate_up [T,2I] (gate | up) -> silu(gate) * up, [T,I]."""
    gu = _f32(gate_up)
    T, I2 = gu.shape
    assert I2 % 2 == 0
    dt, sfx = _real(f32)
    out = np.empty((T, I2 // 2), dtype=dt)
    rc = getattr(lib(), "oracle_swiglu" + sfx)(_p(gu), ctypes.c_int64(T), ctypes.c_int(I2 // 2), _p(out))
    assert rc == 0
    return out


def linear(x, W, f32: bool = False):
    """x [T,K], W [N,K] -> x @ W.T, [T,N]."""
    x, W = _f32(x), _f32(W)
    T, K = x.shape
    N = W.shape[0]
    assert W.shape[1] == K
    dt, sfx = _real(f32)
    y = np.empty((T, N), dtype=dt)
    rc = getattr(lib(), "oracle_linear" + sfx)(_p(x), _p(W), ctypes.c_int64(T), ctypes.c_int(K), ctypes.c_int(N), _p(y))
    assert rc == 0
    return y


def attn_bwd_packed(q, k, v, dout, cu_seqlens, scale: float, f32: bool = False):
    """Backward of attn_packed: q, dout [tot,Hq,d], k, v [tot,Hkv,d] -> (dq, dk, dv)."""
    q, k, v, dout, cu = _f32(q), _f32(k), _f32(v), _f32(dout), _i32(cu_seqlens)
    tot, Hq, d = q.shape
    Hkv = k.shape[1]
    assert dout.shape == q.shape and v.shape == k.shape and cu[-1] == tot
    dt, sfx = _real(f32)
    dq = np.empty((tot, Hq, d), dtype=dt)
    dk = np.empty((tot, Hkv, d), dtype=dt)
    dv = np.empty((tot, Hkv, d), dtype=dt)
    rc = getattr(lib(), "oracle_attn_bwd_packed" + sfx)(
        _p(q), _p(k), _p(v), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(Hq), ctypes.c_int(Hkv),
        ctypes.c_int(d), ctypes.c_double(scale), _p(dq), _p(dk), _p(dv))
    assert rc == 0
    return dq, dk, dv
