"""ctypes front end of the float64 CPU oracle (``diffqkv_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The CUDA library and its Python binding never import
this package; only the test suite, the smoke check and the benchmark's
CPU-baseline leg do.  Nothing here touches CUDA or the product package.

Tensors are numpy arrays in their storage dtype: ``float32``, or ``uint16`` holding
bf16 bit patterns.  Results are ``float64``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "diffqkv_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

BF16, F32 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Cache(C.Structure):
    _fields_ = [
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("k_stride_blk", C.c_int64), ("k_stride_head", C.c_int64), ("k_stride_tok", C.c_int64),
        ("v_stride_blk", C.c_int64), ("v_stride_head", C.c_int64), ("v_stride_tok", C.c_int64),
        ("seqlens", C.c_void_p), ("page_table", C.c_void_p),
        ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_set_threads.restype = C.c_int
        _lib.oracle_decode.restype = C.c_int
        _lib.oracle_decode_splits.restype = C.c_int
        _lib.oracle_prefill.restype = C.c_int
        _lib.oracle_kv_bytes.restype = C.c_double
    return _lib


def set_threads(n: int = 0) -> int:
    """Set (n > 0) and return the number of OpenMP threads the oracle will use."""
    return int(lib().oracle_set_threads(C.c_int(n)))


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle tensors are float32 or uint16 (bf16 bits), got {a.dtype}")


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else C.c_void_p(a.ctypes.data)


@dataclass
class Cache:
    """Host view of a K/V cache.  Strides are in elements; the channel dim is contiguous.

    Contiguous: ``blk`` is the sequence index.  Paged: ``blk`` is the physical page id
    taken from ``page_table[b, j // page_size]`` and the token stride applies to the
    slot ``j % page_size``.
    """
    k: np.ndarray
    v: np.ndarray
    k_strides: Sequence[int]  # (blk, head, tok)
    v_strides: Sequence[int]
    seqlens: np.ndarray        # int32 [batch]
    page_table: Optional[np.ndarray] = None  # int32 [batch, max_pages_per_seq]
    page_size: int = 0

    def c_struct(self) -> _Cache:
        assert self.seqlens.dtype == np.int32 and self.seqlens.flags.c_contiguous
        pt = self.page_table
        if pt is not None:
            assert pt.dtype == np.int32 and pt.flags.c_contiguous and pt.ndim == 2
        return _Cache(
            self.k.ctypes.data, self.v.ctypes.data,
            *[int(s) for s in self.k_strides], *[int(s) for s in self.v_strides],
            self.seqlens.ctypes.data, None if pt is None else pt.ctypes.data,
            int(self.page_size), 0 if pt is None else int(pt.shape[1]))


def decode(q: np.ndarray, cache: Cache, n_q: int, n_k: int, n_v: int, d_qk: int, d_v: int,
           scale: float, pairs: Optional[np.ndarray] = None):
    """DiffQKV decode attention. q [batch, n_q, d_qk]. Returns (out [batch,n_q,d_v], lse [batch,n_q]).

    With ``pairs`` (int32 [n, 2] of (b, h)) only those rows are computed; the rest are NaN.
    """
    dt = _dtype_code(q)
    assert _dtype_code(cache.k) == dt and _dtype_code(cache.v) == dt
    q = np.ascontiguousarray(q)
    batch = q.shape[0]
    out = np.full((batch, n_q, d_v), np.nan, dtype=np.float64)
    lse = np.full((batch, n_q), np.nan, dtype=np.float64)
    cs = cache.c_struct()
    n_pairs = 0
    if pairs is not None:
        pairs = np.ascontiguousarray(pairs, dtype=np.int32)
        n_pairs = pairs.shape[0]
    rc = lib().oracle_decode(_ptr(q), C.byref(cs), batch, n_q, n_k, n_v, d_qk, d_v, dt,
                             C.c_double(scale), _ptr(pairs), n_pairs, _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError("n_k and n_v must divide n_q")
    return out, lse


def decode_topk(q: np.ndarray, cache: Cache, n_q: int, n_k: int, n_v: int, d_qk: int, d_v: int, scale: float,
                topk: int):
    """Selective V fetching: attention over the `topk` highest-scoring cached tokens of every query head only.

    Returns (out [batch,n_q,d_v], lse [batch,n_q], selected [batch,n_q,topk] int32 (-1 padded, best first),
    margin [batch,n_q] = gap between the last kept and the first dropped score)."""
    dt = _dtype_code(q)
    q = np.ascontiguousarray(q)
    batch = q.shape[0]
    out = np.zeros((batch, n_q, d_v), dtype=np.float64)
    lse = np.zeros((batch, n_q), dtype=np.float64)
    sel = np.zeros((batch, n_q, topk), dtype=np.int32)
    margin = np.zeros((batch, n_q), dtype=np.float64)
    cs = cache.c_struct()
    lib().oracle_decode_topk.restype = C.c_int
    rc = lib().oracle_decode_topk(_ptr(q), C.byref(cs), batch, n_q, n_k, n_v, d_qk, d_v, dt, C.c_double(scale),
                                  int(topk), _ptr(out), _ptr(lse), _ptr(sel), _ptr(margin))
    if rc != 0:
        raise ValueError("n_k and n_v must divide n_q and topk must be positive")
    return out, lse, sel, margin


def decode_kup(q: np.ndarray, W_kup: np.ndarray, cache: Cache, n_q: int, n_k: int, n_v: int, d_v: int, scale: float):
    """Decode over keys cached at width d_k < d_q: every cached key goes through the linear layer W_kup[hk]
    ([n_k, d_q, d_k]) before its inner product with the query.  q [batch, n_q, d_q]; returns (out, lse)."""
    dt = _dtype_code(q)
    assert _dtype_code(W_kup) == dt and _dtype_code(cache.k) == dt
    q, W_kup = np.ascontiguousarray(q), np.ascontiguousarray(W_kup)
    batch, _, d_q = q.shape
    assert W_kup.shape[:2] == (n_k, d_q)
    d_k = W_kup.shape[2]
    out = np.zeros((batch, n_q, d_v), dtype=np.float64)
    lse = np.zeros((batch, n_q), dtype=np.float64)
    cs = cache.c_struct()
    lib().oracle_decode_kup.restype = C.c_int
    rc = lib().oracle_decode_kup(_ptr(q), _ptr(W_kup), C.byref(cs), batch, n_q, n_k, n_v, d_q, d_k, d_v, dt,
                                 C.c_double(scale), _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError("n_k and n_v must divide n_q")
    return out, lse


def decode_splits(q: np.ndarray, cache: Cache, n_q: int, n_k: int, n_v: int, d_qk: int, d_v: int,
                  scale: float, cuts: Sequence[int]):
    """Per-split normalised outputs and lse for token ranges [cuts[s], cuts[s+1])."""
    dt = _dtype_code(q)
    q = np.ascontiguousarray(q)
    batch = q.shape[0]
    cuts = np.ascontiguousarray(cuts, dtype=np.int64)
    ns = len(cuts) - 1
    o = np.zeros((batch, n_q, ns, d_v), dtype=np.float64)
    l = np.zeros((batch, n_q, ns), dtype=np.float64)
    cs = cache.c_struct()
    rc = lib().oracle_decode_splits(_ptr(q), C.byref(cs), batch, n_q, n_k, n_v, d_qk, d_v, dt,
                                    C.c_double(scale), _ptr(cuts), ns, _ptr(o), _ptr(l))
    if rc != 0:
        raise ValueError("n_k and n_v must divide n_q")
    return o, l


def combine(o_partial: np.ndarray, lse_partial: np.ndarray):
    """Log-sum-exp merge of per-split partials [..., S, d_v] / [..., S] -> ([..., d_v], [...])."""
    o_partial = np.ascontiguousarray(o_partial, dtype=np.float64)
    lse_partial = np.ascontiguousarray(lse_partial, dtype=np.float64)
    lead = lse_partial.shape[:-1]
    S = lse_partial.shape[-1]
    d_v = o_partial.shape[-1]
    rows = int(np.prod(lead)) if lead else 1
    out = np.zeros(lead + (d_v,), dtype=np.float64)
    lse = np.zeros(lead, dtype=np.float64)
    lib().oracle_combine(_ptr(o_partial), _ptr(lse_partial), C.c_int64(rows), S, d_v, _ptr(out), _ptr(lse))
    return out, lse


def cache_append(k_new: np.ndarray, v_new: np.ndarray, cache: Cache):
    """Write k_new [batch,q_len,n_k,d_qk], v_new [batch,q_len,n_v,d_v] at positions seqlens[b]+i."""
    dt = _dtype_code(k_new)
    k_new = np.ascontiguousarray(k_new)
    v_new = np.ascontiguousarray(v_new)
    batch, q_len, n_k, d_qk = k_new.shape
    _, _, n_v, d_v = v_new.shape
    cs = cache.c_struct()
    lib().oracle_cache_append(_ptr(k_new), _ptr(v_new), q_len, C.byref(cs), batch, n_k, n_v, d_qk, d_v, dt)


def prefill(q: np.ndarray, past: np.ndarray, cache: Cache, n_k: int, n_v: int, d_v: int, scale: float,
            rows: Optional[np.ndarray] = None):
    """Causal attention of q [batch, q_len, n_q, d_qk] over a cache that already holds the new rows.

    Query row i of sequence b sees tokens 0 .. past[b] + i.  With ``rows`` (int32 [n,3] of
    (b, i, h)) returns ([n, d_v], [n]); otherwise ([batch,q_len,n_q,d_v], [batch,q_len,n_q]).
    """
    dt = _dtype_code(q)
    q = np.ascontiguousarray(q)
    batch, q_len, n_q, d_qk = q.shape
    past = np.ascontiguousarray(past, dtype=np.int32)
    cs = cache.c_struct()
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        n_rows = rows.shape[0]
        out = np.zeros((n_rows, d_v), dtype=np.float64)
        lse = np.zeros((n_rows,), dtype=np.float64)
    else:
        n_rows = 0
        out = np.zeros((batch, q_len, n_q, d_v), dtype=np.float64)
        lse = np.zeros((batch, q_len, n_q), dtype=np.float64)
    rc = lib().oracle_prefill(_ptr(q), q_len, _ptr(past), C.byref(cs), batch, n_q, n_k, n_v, d_qk, d_v, dt,
                              C.c_double(scale), _ptr(rows), C.c_int64(n_rows), _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError("n_k and n_v must divide n_q")
    return out, lse


def augq(h: np.ndarray, W_Q: np.ndarray, W_gate: np.ndarray, W_up: np.ndarray, W_down: np.ndarray,
         rows: Optional[np.ndarray] = None):
    """Augmented Q: q = (silu(x Wg^T) * (x Wu^T)) Wd^T with x = h W_Q^T; weights [out, in]."""
    dt = _dtype_code(h)
    arrs = [np.ascontiguousarray(a) for a in (h, W_Q, W_gate, W_up, W_down)]
    h, W_Q, W_gate, W_up, W_down = arrs
    T, d_model = h.shape
    d_q0 = W_Q.shape[0]
    d_aug = W_gate.shape[0]
    d_out = W_down.shape[0]
    assert W_Q.shape == (d_q0, d_model) and W_gate.shape == (d_aug, d_q0)
    assert W_up.shape == (d_aug, d_q0) and W_down.shape == (d_out, d_aug)
    n_rows = 0
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n_rows = rows.shape[0]
    out = np.zeros((n_rows if rows is not None else T, d_out), dtype=np.float64)
    lib().oracle_augq(_ptr(h), _ptr(W_Q), _ptr(W_gate), _ptr(W_up), _ptr(W_down), C.c_int64(T),
                      d_model, d_q0, d_aug, d_out, dt, _ptr(rows), C.c_int64(n_rows), _ptr(out))
    return out


def linear(x: np.ndarray, W: np.ndarray) -> np.ndarray:
    """y = x W^T (W is [out, in], no bias) in float64 from the stored values."""
    dt = _dtype_code(x)
    assert _dtype_code(W) == dt
    x, W = np.ascontiguousarray(x), np.ascontiguousarray(W)
    T, d_in = x.shape
    d_out = W.shape[0]
    assert W.shape == (d_out, d_in)
    y = np.zeros((T, d_out), dtype=np.float64)
    lib().oracle_linear(_ptr(x), _ptr(W), C.c_int64(T), d_in, d_out, dt, _ptr(y))
    return y


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding (rotate-half pairing) of x [T, n_heads, d] float64 at positions pos [T]; returns a copy."""
    y = np.array(x, dtype=np.float64, order="C", copy=True)
    T, n_heads, d = y.shape
    assert d % 2 == 0
    pos = np.ascontiguousarray(pos, dtype=np.int64)
    assert pos.shape == (T,)
    lib().oracle_rope(_ptr(y), _ptr(pos), C.c_int64(T), n_heads, d, C.c_double(theta))
    return y


def rope_tables(pos: np.ndarray, d: int, theta: float):
    """cos and sin of the rotary angles, float64 [T, d/2]: the tables a caller hands to the GPU entry points."""
    i = np.arange(d // 2, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * np.power(float(theta), -2.0 * i / d)[None, :]
    return np.cos(ang), np.sin(ang)


def kv_bytes(seqlens: np.ndarray, n_k: int, n_v: int, d_qk: int, d_v: int, elt_bytes: int) -> float:
    """Bytes of K and V cache the method must stream once (the paper's cache cost model, alpha = element size)."""
    seqlens = np.ascontiguousarray(seqlens, dtype=np.int32)
    return float(lib().oracle_kv_bytes(_ptr(seqlens), len(seqlens), n_k, n_v, d_qk, d_v, elt_bytes))
