"""CPU oracle for the sparse-decode hot path (numpy front end of ``sparse_decode_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only the tests,
the smoke check and the CPU-baseline leg of the benchmark do.  It shares no code with
the CUDA path: inputs arrive as raw bf16 bit patterns (numpy ``uint16``) and integer
tables, and every result is fp64.

The five steps can be called one by one so that each CUDA stage is checkable on its own:

    meta      = quest_meta(...)          page summaries (min / max of K per channel)
    S, P, pr  = quest_scores(...)        per-query-head bound, per-kv-head score, presence
    sel, cnt, theta = topk_pages(...)    k largest, ties to the lower page, ascending order
    out, lse  = attend(...)              softmax attention over the selected tokens
                                         (+ H2O accumulated attention mass, in place)

``decode_step`` chains them the way one decode step of the engine does.  ``h2o_retain`` /
``h2o_compact`` are the consumer of the H2O statistic: the retained set and the eviction.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparse_decode_oracle.c")
_LIB = os.path.join(_HERE, "libsparse_decode_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (``-O2 -fopenmp``, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(build())
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops over (request, kv-head) will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def default_scale(D: int) -> float:
    return 1.0 / float(np.sqrt(float(D)))


def quest_meta(k_cache, page_table, seq_lens, page_size=16, first_tok=None, meta=None):
    """Page summaries.  ``k_cache`` [P,H_kv,p,D] uint16 → ``meta`` [P,H_kv,2,D] uint16
    (row 0 = channel-wise min, row 1 = max over the page's valid tokens).  ``first_tok``
    None → only the page holding each request's newest token; an int array → every page
    from that token on (0 = all).  Pages no request refers to keep their old contents."""
    k_cache = _u16(k_cache)
    P, H_kv, p, D = k_cache.shape
    assert p == page_size
    page_table = _i32(page_table)
    seq_lens = _i32(seq_lens)
    B, max_pages = page_table.shape
    if meta is None:
        meta = np.zeros((P, H_kv, 2, D), dtype=np.uint16)
    else:
        meta = _u16(meta).copy()
    ft = None if first_tok is None else _i32(first_tok)
    _load().se_oracle_meta(B, H_kv, D, p, max_pages,
                           _p(k_cache, ctypes.c_uint16), _p(page_table, ctypes.c_int32),
                           _p(seq_lens, ctypes.c_int32), _p(ft, ctypes.c_int32),
                           _p(meta, ctypes.c_uint16))
    return meta


def quest_scores(q, meta, page_table, seq_lens, page_size=16, sm_scale=None, group_sum=False):
    """Returns (S [B,H_q,max_pages], P [B,H_kv,max_pages], present [B,max_pages] bool)."""
    q = _u16(q)
    meta = _u16(meta)
    B, H_q, D = q.shape
    H_kv = meta.shape[1]
    page_table = _i32(page_table)
    seq_lens = _i32(seq_lens)
    max_pages = page_table.shape[1]
    S = np.zeros((B, H_q, max_pages), dtype=np.float64)
    P = np.zeros((B, H_kv, max_pages), dtype=np.float64)
    present = np.zeros((B, max_pages), dtype=np.uint8)
    scale = default_scale(D) if sm_scale is None else float(sm_scale)
    _load().se_oracle_scores(B, H_q, H_kv, D, page_size, max_pages,
                             ctypes.c_double(scale), int(bool(group_sum)),
                             _p(q, ctypes.c_uint16), _p(meta, ctypes.c_uint16),
                             _p(page_table, ctypes.c_int32), _p(seq_lens, ctypes.c_int32),
                             _p(S, ctypes.c_double), _p(P, ctypes.c_double),
                             _p(present, ctypes.c_uint8))
    return S, P, present.astype(bool)


def topk_pages(P, present, budget, page_size=16, k_max=None, sink_pages=0, recent_pages=0, seq_lens=None):
    """Returns (sel_idx [B,H_kv,k_max] int32 ascending / -1 padded, sel_cnt [B,H_kv],
    theta [B,H_kv,2] = the k_eff-th and (k_eff+1)-th largest candidate score, NaN where
    undefined).  ``sink_pages`` / ``recent_pages`` force the first / last pages of every request
    into the result outside the budget (``seq_lens`` then tells where a request ends)."""
    P = np.ascontiguousarray(P, dtype=np.float64)
    B, H_kv, max_pages = P.shape
    pres = np.ascontiguousarray(present, dtype=np.uint8)
    if k_max is None:
        k_max = max(budget // page_size + sink_pages + recent_pages, 1)
    n_pages = None
    if seq_lens is not None:
        n_pages = np.ascontiguousarray((np.asarray(seq_lens, dtype=np.int64) + page_size - 1) // page_size, dtype=np.int32)
    elif recent_pages:
        raise ValueError("recent_pages needs seq_lens")
    sel_idx = np.full((B, H_kv, k_max), -1, dtype=np.int32)
    sel_cnt = np.zeros((B, H_kv), dtype=np.int32)
    theta = np.zeros((B, H_kv, 2), dtype=np.float64)
    _load().se_oracle_topk(B, H_kv, page_size, max_pages, k_max, int(budget),
                           int(sink_pages), int(recent_pages), _p(n_pages, ctypes.c_int32),
                           _p(P, ctypes.c_double), _p(pres, ctypes.c_uint8),
                           _p(sel_idx, ctypes.c_int32), _p(sel_cnt, ctypes.c_int32),
                           _p(theta, ctypes.c_double))
    return sel_idx, sel_cnt, theta


def attend(q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
           page_size=16, sm_scale=None, u_accum=None):
    """Returns (out [B,H_q,D], lse [B,H_q]); ``u_accum`` [P,H_kv,p] float64 is updated
    in place when given."""
    q = _u16(q)
    k_cache = _u16(k_cache)
    v_cache = _u16(v_cache)
    B, H_q, D = q.shape
    P_, H_kv, p, _ = k_cache.shape
    assert p == page_size
    page_table = _i32(page_table)
    seq_lens = _i32(seq_lens)
    sel_idx = _i32(sel_idx)
    sel_cnt = _i32(sel_cnt)
    max_pages = page_table.shape[1]
    k_max = sel_idx.shape[2]
    out = np.zeros((B, H_q, D), dtype=np.float64)
    lse = np.zeros((B, H_q), dtype=np.float64)
    if u_accum is not None:
        assert u_accum.dtype == np.float64 and u_accum.flags.c_contiguous
        assert u_accum.shape == (P_, H_kv, p)
    scale = default_scale(D) if sm_scale is None else float(sm_scale)
    _load().se_oracle_attend(B, H_q, H_kv, D, p, max_pages, k_max, ctypes.c_double(scale),
                             _p(q, ctypes.c_uint16), _p(k_cache, ctypes.c_uint16),
                             _p(v_cache, ctypes.c_uint16), _p(page_table, ctypes.c_int32),
                             _p(seq_lens, ctypes.c_int32), _p(sel_idx, ctypes.c_int32),
                             _p(sel_cnt, ctypes.c_int32), _p(out, ctypes.c_double),
                             _p(lse, ctypes.c_double), _p(u_accum, ctypes.c_double))
    return out, lse


def h2o_retain(u_accum, page_table, seq_lens, budget, recent, page_size=16):
    """H2O retained set per (request, kv-head): returns (keep_idx [B,H_kv,budget] int32, ascending
    token positions, -1 padded; keep_cnt [B,H_kv]).  ``u_accum`` [P,H_kv,p] float64."""
    u_accum = np.ascontiguousarray(u_accum, dtype=np.float64)
    P_, H_kv, p = u_accum.shape
    assert p == page_size
    page_table = _i32(page_table)
    seq_lens = _i32(seq_lens)
    B, max_pages = page_table.shape
    keep_idx = np.full((B, H_kv, int(budget)), -1, dtype=np.int32)
    keep_cnt = np.zeros((B, H_kv), dtype=np.int32)
    _load().se_oracle_h2o_retain(B, H_kv, p, max_pages, int(budget), int(recent),
                                 _p(u_accum, ctypes.c_double), _p(page_table, ctypes.c_int32),
                                 _p(seq_lens, ctypes.c_int32), _p(keep_idx, ctypes.c_int32),
                                 _p(keep_cnt, ctypes.c_int32))
    return keep_idx, keep_cnt


def h2o_compact(k_cache, v_cache, u_accum, page_table, keep_idx, keep_cnt):
    """Eviction as slot compaction.  Returns new copies (k_cache, v_cache, u_accum, new_lens)."""
    k = _u16(k_cache).copy()
    v = _u16(v_cache).copy()
    u = np.ascontiguousarray(u_accum, dtype=np.float64).copy()
    P_, H_kv, p, D = k.shape
    page_table = _i32(page_table)
    keep_idx = _i32(keep_idx)
    keep_cnt = _i32(keep_cnt)
    B, max_pages = page_table.shape
    budget = keep_idx.shape[2]
    new_lens = np.zeros((B,), dtype=np.int32)
    _load().se_oracle_h2o_compact(B, H_kv, D, p, max_pages, P_, budget, _p(k, ctypes.c_uint16),
                                  _p(v, ctypes.c_uint16), _p(u, ctypes.c_double),
                                  _p(page_table, ctypes.c_int32), _p(keep_idx, ctypes.c_int32),
                                  _p(keep_cnt, ctypes.c_int32), _p(new_lens, ctypes.c_int32))
    return k, v, u, new_lens


def token_scores(q, k_cache, page_table, seq_lens, page_size=16, sm_scale=None):
    """Observation-layer selector: returns (s [B, max_pages*p] = max over query heads of the logit,
    present [B, max_pages*p] bool)."""
    q = _u16(q)
    k_cache = _u16(k_cache)
    B, H_q, D = q.shape
    _, H_kv, p, _ = k_cache.shape
    assert p == page_size
    page_table = _i32(page_table)
    seq_lens = _i32(seq_lens)
    max_pages = page_table.shape[1]
    s = np.zeros((B, max_pages * p), dtype=np.float64)
    present = np.zeros((B, max_pages * p), dtype=np.uint8)
    scale = default_scale(D) if sm_scale is None else float(sm_scale)
    _load().se_oracle_token_scores(B, H_q, H_kv, D, p, max_pages, ctypes.c_double(scale),
                                   _p(q, ctypes.c_uint16), _p(k_cache, ctypes.c_uint16),
                                   _p(page_table, ctypes.c_int32), _p(seq_lens, ctypes.c_int32),
                                   _p(s, ctypes.c_double), _p(present, ctypes.c_uint8))
    return s, present.astype(bool)


def token_topk(s, present, seq_lens, budget, recent=0, n_out=None):
    """Returns (tok_idx [B, n_out] ascending / -1 padded, tok_cnt [B], theta [B])."""
    s = np.ascontiguousarray(s, dtype=np.float64)
    pres = np.ascontiguousarray(present, dtype=np.uint8)
    B, n_max = s.shape
    seq_lens = _i32(seq_lens)
    if n_out is None:
        n_out = int(budget) + int(recent)
    tok_idx = np.full((B, n_out), -1, dtype=np.int32)
    tok_cnt = np.zeros((B,), dtype=np.int32)
    theta = np.zeros((B,), dtype=np.float64)
    _load().se_oracle_token_topk(B, n_max, int(n_out), int(budget), int(recent), _p(s, ctypes.c_double),
                                 _p(pres, ctypes.c_uint8), _p(seq_lens, ctypes.c_int32),
                                 _p(tok_idx, ctypes.c_int32), _p(tok_cnt, ctypes.c_int32),
                                 _p(theta, ctypes.c_double))
    return tok_idx, tok_cnt, theta


def token_attend(q, k_cache, v_cache, page_table, seq_lens, tok_idx, tok_cnt, page_size=16, sm_scale=None):
    """Attention of every query head over one token set per request: (out [B,H_q,D], lse [B,H_q])."""
    q = _u16(q)
    k_cache = _u16(k_cache)
    v_cache = _u16(v_cache)
    B, H_q, D = q.shape
    _, H_kv, p, _ = k_cache.shape
    assert p == page_size
    page_table = _i32(page_table)
    seq_lens = _i32(seq_lens)
    tok_idx = _i32(tok_idx)
    tok_cnt = _i32(tok_cnt)
    max_pages = page_table.shape[1]
    out = np.zeros((B, H_q, D), dtype=np.float64)
    lse = np.zeros((B, H_q), dtype=np.float64)
    scale = default_scale(D) if sm_scale is None else float(sm_scale)
    _load().se_oracle_token_attend(B, H_q, H_kv, D, p, max_pages, tok_idx.shape[1], ctypes.c_double(scale),
                                   _p(q, ctypes.c_uint16), _p(k_cache, ctypes.c_uint16),
                                   _p(v_cache, ctypes.c_uint16), _p(page_table, ctypes.c_int32),
                                   _p(seq_lens, ctypes.c_int32), _p(tok_idx, ctypes.c_int32),
                                   _p(tok_cnt, ctypes.c_int32), _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    return out, lse


def decode_step(q, k_cache, v_cache, page_table, seq_lens, budget, meta=None,
                page_size=16, sm_scale=None, u_accum=None, k_max=None, sink_pages=0, recent_pages=0):
    """One decode step: summary of the newest page, scores, top-k, attention."""
    meta = quest_meta(k_cache, page_table, seq_lens, page_size, first_tok=None, meta=meta)
    S, P, present = quest_scores(q, meta, page_table, seq_lens, page_size, sm_scale)
    sel_idx, sel_cnt, theta = topk_pages(P, present, budget, page_size, k_max, sink_pages, recent_pages, seq_lens)
    out, lse = attend(q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                      page_size, sm_scale, u_accum)
    return dict(meta=meta, S=S, P=P, present=present, sel_idx=sel_idx, sel_cnt=sel_cnt,
                theta=theta, out=out, lse=lse)
