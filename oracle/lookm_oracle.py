"""Python face of the fp64 CPU oracle (test infrastructure only -- never on the product path).

Compiles ``lookm_oracle.c`` with gcc into ``_lookm_oracle.so`` next to this file, loads it with
ctypes and composes its per-step functions into the whole LOOK-M compression of a layer:
scores (Eq. 4) -> window + text prior + Top-N (Eq. 5-8) -> cosine matching (Eq. 9) ->
averaged / pivotal / weighted merging (Eq. 10-12) -> dense cache ordered by position.

Tensors are numpy float32 arrays holding bf16-exact values, laid out [tokens, heads, head_dim].
Heads are independent, so the only parallelism is a thread pool over KV heads (ctypes drops the
GIL during the C call).  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import this module; the CUDA library neither imports it nor shares code with it.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lookm_oracle.c")
_SO = os.path.join(_HERE, "_lookm_oracle.so")
_lib = None
_lock = threading.Lock()

MERGE_AVERAGE, MERGE_PIVOTAL, MERGE_WEIGHTED, MERGE_NONE = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    with _lock:                      # the heads of a layer call in from a thread pool
        return _lib_locked()


def _lib_locked():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp, dp, ip, u8p = (C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_int),
                           C.POINTER(C.c_uint8))
        ll = C.c_longlong
        L.lookm_oracle_scores_head.argtypes = [fp, ll, ll, C.c_int, fp, ll, C.c_int, C.c_int,
                                               C.c_double, C.c_int, dp, dp]
        L.lookm_oracle_scores_head.restype = C.c_int
        L.lookm_oracle_lse_rows.argtypes = [fp, ll, fp, ll, C.c_int, C.c_double, ip, C.c_int, dp]
        L.lookm_oracle_lse_rows.restype = C.c_int
        L.lookm_oracle_select.argtypes = [dp, u8p, C.c_int, C.c_int, C.c_int, C.c_int, ip, ip]
        L.lookm_oracle_select.restype = C.c_int
        L.lookm_oracle_match.argtypes = [fp, ll, C.c_int, ip, C.c_int, ip, C.c_int, ip, dp, dp]
        L.lookm_oracle_match.restype = None
        L.lookm_oracle_argmax_rows.argtypes = [dp, C.c_int, C.c_int, ip, dp]
        L.lookm_oracle_argmax_rows.restype = None
        L.lookm_oracle_merge.argtypes = [fp, ll, C.c_int, ip, C.c_int, ip, C.c_int, ip, dp,
                                         C.c_int, dp]
        L.lookm_oracle_merge.restype = C.c_int
        L.lookm_oracle_decode_head.argtypes = [fp, ll, C.c_int, fp, ll, fp, ll, C.c_int, C.c_int,
                                               C.c_double, dp]
        L.lookm_oracle_decode_head.restype = C.c_int
        _lib = L
    return _lib


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(C.POINTER(t))


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.ndim == 3, "expected [tokens, heads, head_dim]"
    return a


def _head_ptr(a: np.ndarray, head: int):
    """Pointer to a[0, head, 0] of a contiguous [L, H, d] float32 array and its token stride."""
    H, d = a.shape[1], a.shape[2]
    addr = a.ctypes.data + head * d * 4
    return C.cast(addr, C.POINTER(C.c_float)), H * d


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def _pool_map(fn, items, threads):
    items = list(items)
    if threads <= 1 or len(items) <= 1:
        return [fn(it) for it in items]
    with ThreadPoolExecutor(max_workers=min(threads, len(items))) as ex:
        return list(ex.map(fn, items))


# ---------------------------------------------------------------------------------------------
# per-step functions
# ---------------------------------------------------------------------------------------------

def scores(q, k, scale: Optional[float] = None, key_begin: int = 0,
           kv_heads: Optional[Sequence[int]] = None, threads: int = 1, want_lse: bool = False):
    """Cumulative attention scores A_s (Eq. 4), [len(kv_heads), L] float64.

    With want_lse also returns the natural-log row log-sum-exp, [len(kv_heads), group, L].
    """
    q, k = _f32(q), _f32(k)
    L, Hq, d = q.shape
    Hkv = k.shape[1]
    assert Hq % Hkv == 0 and k.shape[0] == L and k.shape[2] == d
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if scale is None else float(scale)
    heads = list(range(Hkv)) if kv_heads is None else list(kv_heads)
    out = np.zeros((len(heads), L), dtype=np.float64)
    lse = np.full((len(heads), G, L), np.nan, dtype=np.float64) if want_lse else None

    def one(idx):
        h = heads[idx]
        qp, qst = _head_ptr(q, h * G)
        kp, kst = _head_ptr(k, h)
        lp = _p(lse[idx], C.c_double) if want_lse else None
        rc = lib().lookm_oracle_scores_head(qp, qst, d, G, kp, kst, L, d, scale, key_begin,
                                            _p(out[idx], C.c_double), lp)
        if rc != 0:
            raise MemoryError("oracle scores")

    _pool_map(one, range(len(heads)), threads)
    return (out, lse) if want_lse else out


def lse_rows(q, k, q_head: int, kv_head: int, rows, scale: Optional[float] = None) -> np.ndarray:
    """Natural-log causal log-sum-exp of the given query rows of one query head."""
    q, k = _f32(q), _f32(k)
    d = q.shape[2]
    scale = 1.0 / math.sqrt(d) if scale is None else float(scale)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    out = np.zeros(len(rows), dtype=np.float64)
    qp, qst = _head_ptr(q, q_head)
    kp, kst = _head_ptr(k, kv_head)
    rc = lib().lookm_oracle_lse_rows(qp, qst, kp, kst, d, scale, _p(rows, C.c_int), len(rows),
                                     _p(out, C.c_double))
    if rc != 0:
        raise MemoryError("oracle lse rows")
    return out


def select(score_row, mask, budget: int, window: int, text_prior: bool = True):
    """Window + text prior + Top-N for one head: (kept, evicted) ascending int32 position arrays.

    text_prior=False ranks the candidates by score alone (Eq. 8 without the boost of Eq. 5)."""
    s = np.ascontiguousarray(score_row, dtype=np.float64)
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    L = s.shape[0]
    assert m.shape[0] == L
    nk = min(budget, L)
    kept = np.zeros(nk, dtype=np.int32)
    ev = np.zeros(L - nk, dtype=np.int32)
    rc = lib().lookm_oracle_select(_p(s, C.c_double), _p(m, C.c_uint8), L, budget, window,
                                   1 if text_prior else 0, _p(kept, C.c_int), _p(ev, C.c_int))
    if rc != nk:
        raise ValueError("oracle select rejected its arguments")
    return kept, ev


def match(k, kv_head: int, kept, evicted, want_matrix: bool = False):
    """Cosine nearest kept key of each evicted key of one head: (assign int32, sim float64[, S])."""
    k = _f32(k)
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    ev = np.ascontiguousarray(evicted, dtype=np.int32)
    assign = np.zeros(len(ev), dtype=np.int32)
    sim = np.zeros(len(ev), dtype=np.float64)
    S = np.zeros((len(ev), len(kept)), dtype=np.float64) if want_matrix else None
    kp, kst = _head_ptr(k, kv_head)
    lib().lookm_oracle_match(kp, kst, k.shape[2], _p(kept, C.c_int), len(kept), _p(ev, C.c_int),
                             len(ev), _p(assign, C.c_int), _p(sim, C.c_double),
                             _p(S, C.c_double) if want_matrix else None)
    return (assign, sim, S) if want_matrix else (assign, sim)


def argmax_rows(sim_matrix):
    """Row argmax (lowest slot on ties) and row maximum of a similarity matrix."""
    S = np.ascontiguousarray(sim_matrix, dtype=np.float64)
    ne, nk = S.shape
    assign = np.zeros(ne, dtype=np.int32)
    sim = np.zeros(ne, dtype=np.float64)
    lib().lookm_oracle_argmax_rows(_p(S, C.c_double), ne, nk, _p(assign, C.c_int), _p(sim, C.c_double))
    return assign, sim


def merge(x, kv_head: int, kept, evicted, assign, sim, mode: int) -> np.ndarray:
    """Merged rows [len(kept), d] (float64) of one head of tensor x (keys or values)."""
    x = _f32(x)
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    ev = np.ascontiguousarray(evicted, dtype=np.int32)
    assign = np.ascontiguousarray(assign, dtype=np.int32)
    sim = np.ascontiguousarray(sim, dtype=np.float64)
    assert len(assign) == len(ev) == len(sim)
    d = x.shape[2]
    out = np.zeros((len(kept), d), dtype=np.float64)
    xp, xst = _head_ptr(x, kv_head)
    rc = lib().lookm_oracle_merge(xp, xst, d, _p(kept, C.c_int), len(kept), _p(ev, C.c_int), len(ev),
                                  _p(assign, C.c_int), _p(sim, C.c_double), int(mode),
                                  _p(out, C.c_double))
    if rc != 0:
        raise MemoryError("oracle merge")
    return out


# ---------------------------------------------------------------------------------------------
# the whole path
# ---------------------------------------------------------------------------------------------

def compress_layer(q, k, v, mask, budget: int, window: int, mode: int,
                   scale: Optional[float] = None, kv_heads: Optional[Sequence[int]] = None,
                   threads: int = 1, score_dtype=np.float64, text_prior: bool = True):
    """Compress one request's layer.  Returns a dict of per-head results for `kv_heads`.

    mode MERGE_NONE evicts without merging (no matching is done: `assign` and `sim` are empty);
    text_prior=False selects by score alone.

    score_dtype=np.float32 rounds the scores to fp32 before selection, and the similarities
    before weighted merging are kept in fp64; this is what a comparison with a kernel that
    decides in fp32 uses.
    """
    q, k, v = _f32(q), _f32(k), _f32(v)
    L = q.shape[0]
    heads = list(range(k.shape[1])) if kv_heads is None else list(kv_heads)
    A = scores(q, k, scale=scale, kv_heads=heads, threads=threads)
    res = {"kv_heads": heads, "scores": A, "kept": [], "evicted": [], "assign": [], "sim": [],
           "out_k": [], "out_v": []}

    def one(idx):
        h = heads[idx]
        srow = A[idx].astype(score_dtype).astype(np.float64)
        kept, ev = select(srow, mask, budget, window, text_prior=text_prior)
        if mode == MERGE_NONE:
            assign, sim = np.zeros(0, dtype=np.int32), np.zeros(0)
            ev_m = ev[:0]
        else:
            assign, sim = match(k, h, kept, ev)
            ev_m = ev
        ok = merge(k, h, kept, ev_m, assign, sim, mode)
        ov = merge(v, h, kept, ev_m, assign, sim, mode)
        return kept, ev, assign, sim, ok, ov

    for kept, ev, assign, sim, ok, ov in _pool_map(one, range(len(heads)), threads):
        res["kept"].append(kept); res["evicted"].append(ev); res["assign"].append(assign)
        res["sim"].append(sim); res["out_k"].append(ok); res["out_v"].append(ov)
    res["out_len"] = min(budget, L)
    return res


def compress_varlen(q, k, v, mask, cu_seqlens, budgets, windows, modes,
                    scale: Optional[float] = None, kv_heads: Optional[Sequence[int]] = None,
                    threads: int = 1, score_dtype=np.float64, text_prior: bool = True):
    """Packed batch: every request compressed on its own slice of the token axis."""
    out = []
    for r in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[r]), int(cu_seqlens[r + 1])
        out.append(compress_layer(q[a:b], k[a:b], v[a:b], mask[a:b], int(budgets[r]),
                                  int(windows[r]), int(modes[r]), scale=scale, kv_heads=kv_heads,
                                  threads=threads, score_dtype=score_dtype, text_prior=text_prior))
    return out


# ---------------------------------------------------------------------------------------------
# the step after the path: token generation over a cache (Section 3.1, Eq. 2-3)
# ---------------------------------------------------------------------------------------------

def decode_step(q_t, k_new, v_new, cache_k, cache_v, scale: Optional[float] = None):
    """One generation step of one layer.

    q_t [Hq, d]; k_new, v_new [Hkv, d]; cache_k, cache_v [Hkv, n, d] (float32 arrays holding the
    cached rows).  The new rows are appended (Eq. 2), then every query head attends over its KV
    head's n + 1 rows (Eq. 3).  Returns (out [Hq, d] float64, cache_k', cache_v' [Hkv, n + 1, d]).
    """
    q_t = np.ascontiguousarray(q_t, dtype=np.float32)
    ck = np.concatenate([np.asarray(cache_k, dtype=np.float32),
                         np.asarray(k_new, dtype=np.float32)[:, None, :]], axis=1)
    cv = np.concatenate([np.asarray(cache_v, dtype=np.float32),
                         np.asarray(v_new, dtype=np.float32)[:, None, :]], axis=1)
    ck, cv = np.ascontiguousarray(ck), np.ascontiguousarray(cv)
    Hq, d = q_t.shape
    Hkv, n, _ = ck.shape
    assert Hq % Hkv == 0
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if scale is None else float(scale)
    out = np.zeros((Hq, d), dtype=np.float64)
    for h in range(Hkv):
        rc = lib().lookm_oracle_decode_head(_p(q_t[h * G:], C.c_float), d, G, _p(ck[h], C.c_float), d,
                                            _p(cv[h], C.c_float), d, n, d, scale,
                                            _p(out[h * G:], C.c_double))
        if rc != 0:
            raise MemoryError("oracle decode")
    return out, ck, cv
