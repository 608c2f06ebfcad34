"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, sizes its workspace, and rejects bad arguments before
launching anything."""
import ctypes
import os
import re

import pytest

from paper_2609_39068_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            src = open(os.path.join(inc, fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(se_[a-z_0-9]+)\s*\(", src))
    return names


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_symbols()
    assert {"se_meta_update", "se_page_select", "se_sparse_decode"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) <= names
    assert lib.se_version() >= 100


def test_strerror_texts():
    assert binding.se_strerror(0) == "ok"
    for code in (-1, -2, -3, -4, -5, -99):
        assert binding.se_strerror(code)


def test_workspace_bytes_is_pure_and_monotone():
    p = binding.make_params(8, 32, 8, 128, 2048, 16384, 128)
    n1 = binding.se_workspace_bytes(p)
    assert n1 > 0 and n1 % 256 == 0 and n1 == binding.se_workspace_bytes(p)
    p2 = binding.make_params(16, 32, 8, 128, 2048, 16384, 128)
    assert binding.se_workspace_bytes(p2) > n1


def test_decode_split_plan():
    # few pairs: split (CTAs per pair, or warps per pair); two or more pairs per SM: no split
    few = binding.make_params(8, 32, 8, 128, 2048, 16384, 128)
    many = binding.make_params(64, 32, 8, 128, 4096, 140000, 128)
    assert binding.se_decode_num_splits(few) == 2                 # 64 pairs: two CTAs per pair
    # 24 pairs: 148 / 24 = 6 CTAs per pair would need 24 clusters of 6 resident at once; only 22 are, so 5
    assert binding.se_decode_num_splits(binding.make_params(3, 32, 8, 128, 2048, 16384, 128)) == 5
    # more requests than the scoring kernel's per-request tables hold: refused as a shape, not at launch
    assert binding.se_workspace_bytes(binding.make_params(8192, 8, 8, 128, 64, 1 << 20, 16)) > 0
    assert binding.se_workspace_bytes(binding.make_params(8193, 8, 8, 128, 64, 1 << 20, 16)) == 0
    assert binding.se_decode_num_splits(binding.make_params(24, 32, 8, 128, 2048, 16384, 128)) == 6   # 192 pairs: warps
    assert binding.se_decode_num_splits(many) == 1
    assert binding.se_decode_num_splits(binding.make_params(8, 32, 8, 96, 2048, 16384, 128)) == 0


@pytest.mark.parametrize("B,H_kv,k_max,budget,h2o,launches", [
    (1, 2, 16, 256, False, 1),        # config 1: one fused kernel per step
    (8, 8, 128, 2048, False, 1),      # config 2
    (4, 8, 256, 4096, True, 1),       # config 4: the H2O update runs in the same kernel
    (1, 1, 4096, 65536, False, 3),    # one pair, 148 CTAs: scoring, attention (top-k in its prologue), merge kernel
    (24, 8, 128, 2048, False, 4),     # 192 pairs: scoring, top-k, warp-split attention, merge
    (64, 8, 128, 2048, False, 3),     # config 3: scoring, top-k, two warps per pair
    (64, 8, 128, 2048, True, 4),      # ... + the H2O epilogue kernel
    (128, 8, 64, 1024, False, 3),     # 1024 pairs: one warp per pair
    (8, 8, 2048, 16 * 2048, False, 3),  # dense layer: summary update, list of all pages, attention
])
def test_step_launch_plan_follows_from_the_shape(B, H_kv, k_max, budget, h2o, launches):
    p = binding.make_params(B, 4 * H_kv, H_kv, 128, 8192 if k_max > 2048 else 2048, 1 << 16, k_max)
    assert binding.se_decode_step_launches(p, budget, h2o) == launches
    assert binding.se_decode_step_launches(p, 8, h2o) == 0                   # budget below one page
    assert binding.se_decode_step_launches(binding.make_params(B, 4 * H_kv, H_kv, 96, 2048, 1 << 16, k_max), budget, h2o) == 0


def test_decode_step_and_probe_reject_bad_arguments_before_launch():
    lib = binding.load()
    p = binding.make_params(2, 32, 8, 128, 64, 128, 16)
    pp = ctypes.byref(p)
    ok, odd = ctypes.c_void_p(4096), ctypes.c_void_p(4100)
    args = [pp, ok, ok, ok, ok, ok, ok, 256, ok, ok, ok, ok, None, ok, None]
    bad = list(args); bad[4] = None
    assert lib.se_decode_step(*bad) == -3                                     # meta missing
    bad = list(args); bad[10] = odd
    assert lib.se_decode_step(*bad) == -4
    bad = list(args); bad[7] = 8
    assert lib.se_decode_step(*bad) == -1                                     # budget below one page
    bad = list(args); bad[7] = 16 * 17
    assert lib.se_decode_step(*bad) == -1                                     # more pages than k_max
    assert lib.se_probe_gather(None, None, ok, 16, 512, 16, 2, 4, 3, None) == -3
    assert lib.se_probe_gather(ok, None, ok, 16, 500, 16, 2, 4, 3, None) == -1   # piece size not a multiple of 16
    assert lib.se_probe_gather(ok, None, ok, 16, 4096, 32, 8, 8, 1, None) == -1  # does not fit shared memory
    assert lib.se_probe_gather(ok, None, odd, 16, 512, 16, 2, 4, 3, None) == -4


@pytest.mark.parametrize("kw", [
    dict(D=96), dict(page_size=32), dict(H_q=36), dict(H_q=72), dict(B=0), dict(k_max=0),
    dict(k_max=5000), dict(max_pages=0), dict(num_phys_pages=0), dict(sm_scale=-1.0),
])
def test_invalid_params_are_rejected(kw):
    base = dict(B=2, H_q=32, H_kv=8, D=128, max_pages=64, num_phys_pages=128, k_max=16, sm_scale=0.0,
                page_size=16)
    base.update(kw)
    p = binding.make_params(**base)
    assert binding.se_workspace_bytes(p) == 0
    lib = binding.load()
    fake = ctypes.c_void_p(4096)
    rc = lib.se_meta_update(ctypes.byref(p), fake, fake, fake, None, fake, None)
    assert rc in (-1, -2)


def test_null_and_misaligned_pointers_are_rejected_before_launch():
    lib = binding.load()
    p = binding.make_params(2, 32, 8, 128, 64, 128, 16)
    ok = ctypes.c_void_p(4096)
    odd = ctypes.c_void_p(4100)
    assert lib.se_meta_update(ctypes.byref(p), None, ok, ok, None, ok, None) == -3
    assert lib.se_meta_update(ctypes.byref(p), odd, ok, ok, None, ok, None) == -4
    assert lib.se_page_select(ctypes.byref(p), ok, ok, ok, ok, 256, ok, ok, None, None) == -3
    assert lib.se_page_select(ctypes.byref(p), ok, ok, ok, ok, 8, ok, ok, ok, None) == -1      # budget < one page
    assert lib.se_page_select(ctypes.byref(p), ok, ok, ok, ok, 16 * 17, ok, ok, ok, None) == -1  # budget > k_max pages
    assert lib.se_sparse_decode(ctypes.byref(p), ok, ok, ok, ok, ok, ok, ok, ok, None, None, ok, None) == -3
    assert lib.se_sparse_decode(ctypes.byref(p), ok, ok, ok, ok, ok, ok, ok, ok, ok, odd, ok, None) == -4
    assert lib.se_workspace_init(None, ok, None) == -3


def test_h2o_and_token_calls_reject_bad_arguments_before_launch():
    lib = binding.load()
    p = binding.make_params(2, 32, 8, 128, 64, 128, 16)
    pp = ctypes.byref(p)
    ok, odd = ctypes.c_void_p(4096), ctypes.c_void_p(4100)
    # H2O retention / eviction
    assert lib.se_h2o_retain(pp, None, ok, ok, 64, 8, ok, ok, ok, None) == -3
    assert lib.se_h2o_retain(pp, ok, ok, ok, 0, 8, ok, ok, ok, None) == -1          # empty budget
    assert lib.se_h2o_retain(pp, ok, ok, ok, 64, -1, ok, ok, ok, None) == -1
    assert lib.se_h2o_retain(pp, ok, ok, ok, 64, 8, odd, ok, ok, None) == -4
    assert lib.se_h2o_compact(pp, ok, ok, ok, ok, ok, ok, 64, None, ok, None) == -3
    assert lib.se_h2o_compact(pp, ok, odd, ok, ok, ok, ok, 64, ok, ok, None) == -4
    assert lib.se_h2o_compact(pp, ok, ok, ok, ok, ok, ok, 0, ok, ok, None) == -1
    # selection reuse
    assert lib.se_observe_decode(pp, ok, ok, ok, ok, ok, ok, ok, ok, ok, None, ok, None) == -3
    assert lib.se_token_select(pp, ok, ok, 32, 8, ok, ok, 32, ok, None) == -1        # budget + recent > row length
    assert lib.se_token_select(pp, ok, ok, 32, 8, ok, None, 40, ok, None) == -3
    assert lib.se_token_decode(pp, ok, ok, ok, ok, ok, ok, ok, 16 * 16 + 1, ok, ok, ok, None) == -1   # > k_max tiles
    assert lib.se_token_decode(pp, ok, ok, ok, ok, ok, ok, ok, 64, ok, odd, ok, None) == -4
    bad = binding.make_params(2, 32, 8, 96, 64, 128, 16)
    assert lib.se_token_decode(ctypes.byref(bad), ok, ok, ok, ok, ok, ok, ok, 64, ok, ok, ok, None) in (-1, -2)
