"""Thin ctypes binding of ``libsparse_engine.so`` (see ``include/sparse_engine.h``).

Argument marshalling only: every function takes torch CUDA tensors, checks dtype,
contiguity and shape, and passes raw device pointers plus the current CUDA stream to
the C entry point of the same name.  There is no CPU or PyTorch fallback: if the shared
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import _build

SE_OK = 0
SE_DEV_BAD_PAGE_ID = 1
SE_DEV_BAD_SELECTION = 2
SE_DEV_WAIT_TIMEOUT = 4

EXPORTS = ("se_version", "se_strerror", "se_workspace_bytes", "se_decode_num_splits", "se_workspace_init",
           "se_meta_update",
           "se_page_select", "se_page_select_scores", "se_page_select_topk", "se_page_select_fused", "se_sparse_decode", "se_sparse_decode_splits", "se_combine",
           "se_last_device_status", "se_h2o_retain", "se_h2o_compact", "se_observe_decode", "se_token_select",
           "se_token_decode",
           "se_page_select_static", "se_decode_step", "se_decode_step_launches", "se_probe_gather")
SE_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


class SeParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H_q", ctypes.c_int32), ("H_kv", ctypes.c_int32),
                ("D", ctypes.c_int32), ("page_size", ctypes.c_int32), ("max_pages", ctypes.c_int32),
                ("num_phys_pages", ctypes.c_int32), ("k_max", ctypes.c_int32),
                ("sm_scale", ctypes.c_float), ("flags", ctypes.c_uint32),
                ("sink_pages", ctypes.c_int32), ("recent_pages", ctypes.c_int32)]


class SparseEngineError(RuntimeError):
    pass


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True):
    """Loads the shared library (building it with nvcc first if it is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing and _build.needs_build():
        _build.build()
    if not os.path.exists(_build.LIB):
        raise SparseEngineError("libsparse_engine.so is missing; run `python -m paper_2609_39068_b200._build`")
    lib = ctypes.CDLL(_build.LIB)
    vp, i32p, fp = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    pp = ctypes.POINTER(SeParams)
    lib.se_version.restype = ctypes.c_int
    lib.se_strerror.restype = ctypes.c_char_p
    lib.se_strerror.argtypes = [ctypes.c_int]
    lib.se_workspace_bytes.restype = ctypes.c_size_t
    lib.se_workspace_bytes.argtypes = [pp]
    lib.se_decode_num_splits.argtypes = [pp]
    lib.se_workspace_init.argtypes = [pp, vp, vp]
    lib.se_meta_update.argtypes = [pp, vp, i32p, i32p, i32p, vp, vp]
    lib.se_page_select.argtypes = [pp, vp, vp, i32p, i32p, ctypes.c_int32, i32p, i32p, vp, vp]
    lib.se_page_select_scores.argtypes = lib.se_page_select.argtypes
    lib.se_page_select_topk.argtypes = lib.se_page_select.argtypes
    lib.se_page_select_fused.argtypes = [pp, vp, vp, vp, i32p, i32p, ctypes.c_int32, i32p, i32p, vp, vp]
    lib.se_sparse_decode.argtypes = [pp, vp, vp, vp, i32p, i32p, i32p, i32p, fp, fp, fp, vp, vp]
    lib.se_sparse_decode_splits.argtypes = lib.se_sparse_decode.argtypes
    lib.se_combine.argtypes = lib.se_sparse_decode.argtypes
    lib.se_last_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
    lib.se_observe_decode.argtypes = [pp, vp, vp, vp, i32p, i32p, i32p, i32p, fp, fp, vp, vp, vp]
    lib.se_token_select.argtypes = [pp, vp, i32p, ctypes.c_int32, ctypes.c_int32, i32p, i32p, ctypes.c_int32, vp, vp]
    lib.se_token_decode.argtypes = [pp, vp, vp, vp, i32p, i32p, i32p, i32p, ctypes.c_int32, fp, fp, vp, vp]
    lib.se_h2o_retain.argtypes = [pp, fp, i32p, i32p, ctypes.c_int32, ctypes.c_int32, i32p, i32p, vp, vp]
    lib.se_h2o_compact.argtypes = [pp, vp, vp, fp, i32p, i32p, i32p, ctypes.c_int32, i32p, vp, vp]
    lib.se_page_select_static.argtypes = [pp, vp, vp, i32p, i32p, ctypes.c_int32, i32p, i32p, i32p, vp]
    lib.se_decode_step.argtypes = [pp, vp, vp, vp, vp, i32p, i32p, ctypes.c_int32, i32p, i32p, fp, fp, fp, vp, vp]
    lib.se_decode_step_launches.argtypes = [pp, ctypes.c_int32, ctypes.c_int]
    lib.se_probe_gather.argtypes = [vp, vp, i32p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                    ctypes.c_int32, ctypes.c_int32, vp]
    lib.se_probe_gather.restype = ctypes.c_int
    for name in ("se_workspace_init", "se_meta_update", "se_page_select", "se_page_select_fused",
                 "se_sparse_decode", "se_sparse_decode_splits", "se_combine", "se_last_device_status",
                 "se_h2o_retain", "se_h2o_compact", "se_decode_num_splits", "se_page_select_static",
                 "se_observe_decode", "se_token_select", "se_token_decode", "se_page_select_scores",
                 "se_page_select_topk", "se_decode_step", "se_decode_step_launches"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != SE_OK:
        raise SparseEngineError("%s failed: %s (%d)" % (what, load().se_strerror(rc).decode(), rc))


def _ptr(t: Optional[torch.Tensor], dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise SparseEngineError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype:
        raise SparseEngineError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    if not t.is_contiguous():
        raise SparseEngineError("%s must be contiguous" % name)
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_params(B, H_q, H_kv, D, max_pages, num_phys_pages, k_max, sm_scale=0.0, page_size=16,
                sink_pages=0, recent_pages=0, flags=0) -> SeParams:
    return SeParams(B, H_q, H_kv, D, page_size, max_pages, num_phys_pages, k_max, float(sm_scale), int(flags),
                    int(sink_pages), int(recent_pages))


def se_version() -> int:
    return load().se_version()


def se_strerror(code: int) -> str:
    return load().se_strerror(code).decode()


def se_workspace_bytes(p: SeParams) -> int:
    return int(load().se_workspace_bytes(ctypes.byref(p)))


def se_decode_num_splits(p: SeParams) -> int:
    return int(load().se_decode_num_splits(ctypes.byref(p)))


def se_workspace_init(p: SeParams, workspace: torch.Tensor) -> None:
    _check(load().se_workspace_init(ctypes.byref(p), _ptr(workspace, torch.uint8, "workspace"), _stream()),
           "se_workspace_init")


def alloc_workspace(p: SeParams, device="cuda") -> torch.Tensor:
    """Allocates (through torch) and initialises a workspace for ``p``."""
    n = se_workspace_bytes(p)
    if n == 0:
        raise SparseEngineError("invalid se_params")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    se_workspace_init(p, ws)
    return ws


def se_meta_update(p, k_cache, page_table, seq_lens, meta, first_tok=None) -> None:
    _check(load().se_meta_update(ctypes.byref(p), _ptr(k_cache, torch.bfloat16, "k_cache"),
                                 _ptr(page_table, torch.int32, "page_table"),
                                 _ptr(seq_lens, torch.int32, "seq_lens"),
                                 _ptr(first_tok, torch.int32, "first_tok"),
                                 _ptr(meta, torch.bfloat16, "meta"), _stream()), "se_meta_update")


def se_page_select(p, q, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt, workspace,
                   entry="se_page_select") -> None:
    _check(getattr(load(), entry)(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                 _ptr(meta, torch.bfloat16, "meta"),
                                 _ptr(page_table, torch.int32, "page_table"),
                                 _ptr(seq_lens, torch.int32, "seq_lens"), int(budget_tokens),
                                 _ptr(sel_idx, torch.int32, "sel_idx"), _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                 _ptr(workspace, torch.uint8, "workspace"), _stream()), entry)


def se_page_select_scores(*args, **kw) -> None:
    se_page_select(*args, entry="se_page_select_scores", **kw)


def page_scores_view(p: SeParams, workspace: torch.Tensor) -> torch.Tensor:
    """The fp32 page scores the scoring kernel left in ``workspace`` as a [B, H_kv, max_pages] view
    (they follow the control block: byte offset 256 + 8*B*H_kv rounded up to 256; rows of max_pages
    rounded up to a multiple of 4 floats; entries past a request's last page are not written)."""
    pitch = (p.max_pages + 3) // 4 * 4
    n = p.B * p.H_kv * pitch
    off = 256 + (8 * p.B * p.H_kv + 255) // 256 * 256
    flat = workspace[off:off + 4 * n].view(torch.float32)
    return flat.view(p.B, p.H_kv, pitch)[:, :, :p.max_pages]


def se_page_select_fused(p, q, k_cache, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt,
                         workspace) -> None:
    _check(load().se_page_select_fused(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                       _ptr(k_cache, torch.bfloat16, "k_cache"),
                                       _ptr(meta, torch.bfloat16, "meta"),
                                       _ptr(page_table, torch.int32, "page_table"),
                                       _ptr(seq_lens, torch.int32, "seq_lens"), int(budget_tokens),
                                       _ptr(sel_idx, torch.int32, "sel_idx"),
                                       _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                       _ptr(workspace, torch.uint8, "workspace"), _stream()),
           "se_page_select_fused")


def se_sparse_decode(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, lse,
                     workspace, score_accum=None, entry="se_sparse_decode") -> None:
    _check(getattr(load(), entry)(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                   _ptr(k_cache, torch.bfloat16, "k_cache"),
                                   _ptr(v_cache, torch.bfloat16, "v_cache"),
                                   _ptr(page_table, torch.int32, "page_table"),
                                   _ptr(seq_lens, torch.int32, "seq_lens"),
                                   _ptr(sel_idx, torch.int32, "sel_idx"), _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                   _ptr(out, torch.float32, "out"), _ptr(lse, torch.float32, "lse"),
                                   _ptr(score_accum, torch.float32, "score_accum"),
                                   _ptr(workspace, torch.uint8, "workspace"), _stream()), entry)


def se_sparse_decode_splits(*args, **kw) -> None:
    se_sparse_decode(*args, entry="se_sparse_decode_splits", **kw)


def se_combine(*args, **kw) -> None:
    se_sparse_decode(*args, entry="se_combine", **kw)


def se_decode_step(p, q, k_cache, v_cache, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt, out, lse,
                   workspace, score_accum=None) -> None:
    _check(load().se_decode_step(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                 _ptr(k_cache, torch.bfloat16, "k_cache"), _ptr(v_cache, torch.bfloat16, "v_cache"),
                                 _ptr(meta, torch.bfloat16, "meta"), _ptr(page_table, torch.int32, "page_table"),
                                 _ptr(seq_lens, torch.int32, "seq_lens"), int(budget_tokens),
                                 _ptr(sel_idx, torch.int32, "sel_idx"), _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                 _ptr(out, torch.float32, "out"), _ptr(lse, torch.float32, "lse"),
                                 _ptr(score_accum, torch.float32, "score_accum"),
                                 _ptr(workspace, torch.uint8, "workspace"), _stream()), "se_decode_step")


def se_decode_step_launches(p: SeParams, budget_tokens: int, with_score_accum: bool) -> int:
    return int(load().se_decode_step_launches(ctypes.byref(p), int(budget_tokens), int(bool(with_score_accum))))


def se_probe_gather(base0, piece_idx, piece_bytes, pieces_per_stage, stages_per_warp, warps_per_cta, ctas_per_sm,
                    base1=None) -> None:
    """Read-only gather of the pieces ``piece_idx`` (int32 CUDA tensor) of ``base0`` (any CUDA tensor; odd
    lanes read ``base1`` when given) with the given pipeline shape; see the header."""
    for t in (base0, base1, piece_idx):
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise SparseEngineError("se_probe_gather needs contiguous CUDA tensors")
    if piece_idx.dtype != torch.int32:
        raise SparseEngineError("piece_idx must be int32")
    _check(load().se_probe_gather(ctypes.c_void_p(base0.data_ptr()),
                                  None if base1 is None else ctypes.c_void_p(base1.data_ptr()),
                                  ctypes.c_void_p(piece_idx.data_ptr()), int(piece_idx.numel()), int(piece_bytes),
                                  int(pieces_per_stage), int(stages_per_warp), int(warps_per_cta), int(ctas_per_sm),
                                  _stream()), "se_probe_gather")


def se_page_select_static(p, q, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt,
                          dev_status=None) -> None:
    """Page selection that uses the library's built-in scratch array instead of a workspace
    (for callers that cannot allocate); ``dev_status`` is an optional 1-element int32 CUDA
    tensor that receives the call's status word."""
    _check(load().se_page_select_static(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                        _ptr(meta, torch.bfloat16, "meta"),
                                        _ptr(page_table, torch.int32, "page_table"),
                                        _ptr(seq_lens, torch.int32, "seq_lens"), int(budget_tokens),
                                        _ptr(sel_idx, torch.int32, "sel_idx"),
                                        _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                        _ptr(dev_status, torch.int32, "dev_status"), _stream()),
           "se_page_select_static")


def se_observe_decode(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, lse, tok_keys,
                      workspace) -> None:
    _check(load().se_observe_decode(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                    _ptr(k_cache, torch.bfloat16, "k_cache"), _ptr(v_cache, torch.bfloat16, "v_cache"),
                                    _ptr(page_table, torch.int32, "page_table"), _ptr(seq_lens, torch.int32, "seq_lens"),
                                    _ptr(sel_idx, torch.int32, "sel_idx"), _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                    _ptr(out, torch.float32, "out"), _ptr(lse, torch.float32, "lse"),
                                    _ptr(tok_keys, torch.int32, "tok_keys"),
                                    _ptr(workspace, torch.uint8, "workspace"), _stream()), "se_observe_decode")


def se_token_select(p, tok_keys, seq_lens, budget_tokens, recent_tokens, tok_idx, tok_cnt, workspace) -> None:
    _check(load().se_token_select(ctypes.byref(p), _ptr(tok_keys, torch.int32, "tok_keys"),
                                  _ptr(seq_lens, torch.int32, "seq_lens"), int(budget_tokens), int(recent_tokens),
                                  _ptr(tok_idx, torch.int32, "tok_idx"), _ptr(tok_cnt, torch.int32, "tok_cnt"),
                                  int(tok_idx.shape[-1]), _ptr(workspace, torch.uint8, "workspace"), _stream()),
           "se_token_select")


def se_token_decode(p, q, k_cache, v_cache, page_table, seq_lens, tok_idx, tok_cnt, out, lse, workspace) -> None:
    _check(load().se_token_decode(ctypes.byref(p), _ptr(q, torch.bfloat16, "q"),
                                  _ptr(k_cache, torch.bfloat16, "k_cache"), _ptr(v_cache, torch.bfloat16, "v_cache"),
                                  _ptr(page_table, torch.int32, "page_table"), _ptr(seq_lens, torch.int32, "seq_lens"),
                                  _ptr(tok_idx, torch.int32, "tok_idx"), _ptr(tok_cnt, torch.int32, "tok_cnt"),
                                  int(tok_idx.shape[-1]), _ptr(out, torch.float32, "out"),
                                  _ptr(lse, torch.float32, "lse"), _ptr(workspace, torch.uint8, "workspace"),
                                  _stream()), "se_token_decode")


def keys_to_scores(tok_keys):
    """Inverse of the order-preserving integer image used by se_observe_decode: int32 tensor of keys ->
    (float32 scores, bool attended)."""
    k = tok_keys.to(torch.int64) & 0xFFFFFFFF
    bits = torch.where(k >= 0x80000000, k & 0x7FFFFFFF, (~k) & 0xFFFFFFFF)
    bits = torch.where(bits >= 0x80000000, bits - (1 << 32), bits).to(torch.int32)
    return bits.view(torch.float32), k != 0


def se_h2o_retain(p, score_accum, page_table, seq_lens, budget_tokens, recent_tokens, keep_idx, keep_cnt,
                  workspace) -> None:
    _check(load().se_h2o_retain(ctypes.byref(p), _ptr(score_accum, torch.float32, "score_accum"),
                                _ptr(page_table, torch.int32, "page_table"),
                                _ptr(seq_lens, torch.int32, "seq_lens"), int(budget_tokens), int(recent_tokens),
                                _ptr(keep_idx, torch.int32, "keep_idx"), _ptr(keep_cnt, torch.int32, "keep_cnt"),
                                _ptr(workspace, torch.uint8, "workspace"), _stream()), "se_h2o_retain")


def se_h2o_compact(p, k_cache, v_cache, score_accum, page_table, keep_idx, keep_cnt, new_seq_lens,
                   workspace) -> None:
    _check(load().se_h2o_compact(ctypes.byref(p), _ptr(k_cache, torch.bfloat16, "k_cache"),
                                 _ptr(v_cache, torch.bfloat16, "v_cache"),
                                 _ptr(score_accum, torch.float32, "score_accum"),
                                 _ptr(page_table, torch.int32, "page_table"),
                                 _ptr(keep_idx, torch.int32, "keep_idx"), _ptr(keep_cnt, torch.int32, "keep_cnt"),
                                 int(keep_idx.shape[-1]), _ptr(new_seq_lens, torch.int32, "new_seq_lens"),
                                 _ptr(workspace, torch.uint8, "workspace"), _stream()), "se_h2o_compact")


def se_last_device_status(workspace) -> int:
    word = ctypes.c_int32(0)
    _check(load().se_last_device_status(_ptr(workspace, torch.uint8, "workspace"), _stream(),
                                        ctypes.byref(word)), "se_last_device_status")
    return int(word.value)


class DecodeState:
    """Buffers of one layer's decode step for a fixed shape: params, workspace, summaries,
    selection and outputs.  Convenience for tests, the smoke check and the benchmark."""

    def __init__(self, w, k_max: Optional[int] = None, sm_scale: float = 0.0, sink_pages: int = 0,
                 recent_pages: int = 0, workspace: Optional[torch.Tensor] = None, flags: int = 0):
        dev = w.q.device
        self.w = w
        self.k_max = int(k_max if k_max is not None else max(w.budget // 16 + sink_pages + recent_pages, 1))
        self.p = make_params(w.B, w.H_q, w.H_kv, w.D, w.max_pages, w.num_phys_pages, self.k_max, sm_scale,
                             sink_pages=sink_pages, recent_pages=recent_pages, flags=flags)
        # layers of one model step may share a workspace (their calls are ordered on one stream)
        if workspace is not None and workspace.numel() < se_workspace_bytes(self.p):
            raise SparseEngineError("shared workspace is smaller than se_workspace_bytes")
        self.workspace = alloc_workspace(self.p, dev) if workspace is None else workspace
        self.meta = torch.zeros((w.num_phys_pages, w.H_kv, 2, w.D), dtype=torch.bfloat16, device=dev)
        self.sel_idx = torch.full((w.B, w.H_kv, self.k_max), -7, dtype=torch.int32, device=dev)
        self.sel_cnt = torch.full((w.B, w.H_kv), -7, dtype=torch.int32, device=dev)
        self.out = torch.full((w.B, w.H_q, w.D), float("nan"), dtype=torch.float32, device=dev)
        self.lse = torch.full((w.B, w.H_q), float("nan"), dtype=torch.float32, device=dev)

    def rebuild_meta(self):
        ft = torch.zeros(self.w.B, dtype=torch.int32, device=self.w.q.device)
        se_meta_update(self.p, self.w.k_cache, self.w.page_table, self.w.seq_lens, self.meta, first_tok=ft)

    def update_meta(self):
        se_meta_update(self.p, self.w.k_cache, self.w.page_table, self.w.seq_lens, self.meta)

    def select(self, budget: Optional[int] = None, entry="se_page_select"):
        se_page_select(self.p, self.w.q, self.meta, self.w.page_table, self.w.seq_lens,
                       self.w.budget if budget is None else budget, self.sel_idx, self.sel_cnt, self.workspace,
                       entry=entry)

    def decode(self, score_accum=None, entry="se_sparse_decode"):
        se_sparse_decode(self.p, self.w.q, self.w.k_cache, self.w.v_cache, self.w.page_table,
                         self.w.seq_lens, self.sel_idx, self.sel_cnt, self.out, self.lse,
                         self.workspace, score_accum=score_accum, entry=entry)

    def select_fused(self, budget: Optional[int] = None):
        se_page_select_fused(self.p, self.w.q, self.w.k_cache, self.meta, self.w.page_table, self.w.seq_lens,
                             self.w.budget if budget is None else budget, self.sel_idx, self.sel_cnt,
                             self.workspace)

    def step(self, score_accum=None, fused: bool = True, budget: Optional[int] = None):
        """One decode step of the layer: newest-page summary, selection, attention.  ``fused`` =
        se_decode_step (one call, launch plan picked by the library); otherwise the three separate
        calls se_meta_update, se_page_select, se_sparse_decode."""
        if fused:
            se_decode_step(self.p, self.w.q, self.w.k_cache, self.w.v_cache, self.meta, self.w.page_table,
                           self.w.seq_lens, self.w.budget if budget is None else budget, self.sel_idx,
                           self.sel_cnt, self.out, self.lse, self.workspace, score_accum=score_accum)
        else:
            self.update_meta()
            self.select(budget)
            self.decode(score_accum)

    def status(self) -> int:
        return se_last_device_status(self.workspace)
