"""se_page_select_static: the page selection for hosts that cannot allocate device memory
(a serving loop whose pool is already handed out, a plug-in without an allocator, a thread that
must not hit cudaMalloc's implicit synchronisation).  Its score scratch is a fixed array inside
the library, so the call takes no workspace.  It must return exactly what se_page_select
returns, on a first call and on the calls after it (the array keeps old contents), and must
refuse shapes that do not fit the array.  Collected last on purpose."""
import ctypes

import pytest
import torch

from paper_2609_39068_b200 import binding
from paper_2609_39068_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _case(seed, seq, budget, sink_pages=0, recent_pages=0, k_max=None, **kw):
    w = wl.build("noalloc", 990 + seed, 0, seq, 8, 2, 128, budget, "cpu", **kw).to("cuda")
    st = binding.DecodeState(w, sink_pages=sink_pages, recent_pages=recent_pages, k_max=k_max)
    st.rebuild_meta()
    st.select()
    torch.cuda.synchronize()
    return w, st


def test_static_selection_matches_workspace_selection_on_consecutive_calls():
    cases = [
        _case(1, [5000, 3000, 9000, 17], 1024, permute_pool=True, prune_fraction=0.2),
        _case(2, [700, 0, 64, 2049], 256, permute_pool=True, poison_tail=True),   # smaller: stale scores stay behind
        _case(4, [2000, 50, 333, 1], 128, sink_pages=2, recent_pages=3, permute_pool=True),   # forced pages
        _case(5, [300, 33, 1200], 16 * 75, k_max=75, prune_fraction=0.3),         # dense-layer mode: every present page
    ]
    for rep in range(2):                       # two passes: every call after the first meets old contents
        for w, st in cases:
            sel = torch.full_like(st.sel_idx, -9)
            cnt = torch.full_like(st.sel_cnt, -9)
            status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
            binding.se_page_select_static(st.p, w.q, st.meta, w.page_table, w.seq_lens, w.budget, sel, cnt, status)
            torch.cuda.synchronize()
            assert torch.equal(sel, st.sel_idx), "selected pages differ from se_page_select"
            assert torch.equal(cnt, st.sel_cnt)
            assert int(status.item()) == 0
    # the status pointer is optional
    w, st = cases[0]
    sel = torch.full_like(st.sel_idx, -9)
    cnt = torch.full_like(st.sel_cnt, -9)
    binding.se_page_select_static(st.p, w.q, st.meta, w.page_table, w.seq_lens, w.budget, sel, cnt)
    torch.cuda.synchronize()
    assert torch.equal(sel, st.sel_idx) and torch.equal(cnt, st.sel_cnt)


def test_static_selection_reports_a_bad_page_id_through_dev_status():
    w, st = _case(6, [500, 90], 64)
    w.page_table[0, 3] = w.num_phys_pages + 5            # outside the pool: skipped and reported
    st.select()
    torch.cuda.synchronize()
    assert st.status() & binding.SE_DEV_BAD_PAGE_ID
    for rep in range(2):
        sel, cnt = torch.full_like(st.sel_idx, -9), torch.full_like(st.sel_cnt, -9)
        status = torch.zeros((1,), dtype=torch.int32, device="cuda")
        binding.se_page_select_static(st.p, w.q, st.meta, w.page_table, w.seq_lens, w.budget, sel, cnt, status)
        torch.cuda.synchronize()
        assert int(status.item()) & binding.SE_DEV_BAD_PAGE_ID
        assert torch.equal(sel, st.sel_idx) and torch.equal(cnt, st.sel_cnt)
    # and a clean call afterwards reports a clean status again
    w.page_table[0, 3] = 3
    sel, cnt = torch.full_like(st.sel_idx, -9), torch.full_like(st.sel_cnt, -9)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    binding.se_page_select_static(st.p, w.q, st.meta, w.page_table, w.seq_lens, w.budget, sel, cnt, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0


def test_static_selection_rejects_what_does_not_fit():
    lib = binding.load()
    w, st = _case(3, [100], 64)
    too_big = binding.make_params(64, 32, 8, 128, 4096, 1 << 18, 128)       # 8 MiB of scores
    assert 256 + 4 * 64 * 8 * 4096 > binding.SE_STATIC_SCRATCH_BYTES
    ptr = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = lib.se_page_select_static(ctypes.byref(too_big), ptr(w.q), ptr(st.meta), ptr(w.page_table),
                                   ptr(w.seq_lens), 2048, ptr(st.sel_idx), ptr(st.sel_cnt), None, None)
    assert rc == -6 and "scratch" in binding.se_strerror(rc)
    rc = lib.se_page_select_static(ctypes.byref(st.p), ptr(w.q), ptr(st.meta), ptr(w.page_table),
                                   ptr(w.seq_lens), 8, ptr(st.sel_idx), ptr(st.sel_cnt), None, None)
    assert rc == -1                                                          # budget below one page
    rc = lib.se_page_select_static(ctypes.byref(st.p), None, ptr(st.meta), ptr(w.page_table),
                                   ptr(w.seq_lens), 64, ptr(st.sel_idx), ptr(st.sel_cnt), None, None)
    assert rc == -3
    # a bad shape gets the code every other entry point returns for it
    bad_d = binding.make_params(1, 8, 2, 96, 8, 8, 4)
    rc = lib.se_page_select_static(ctypes.byref(bad_d), ptr(w.q), ptr(st.meta), ptr(w.page_table),
                                   ptr(w.seq_lens), 64, ptr(st.sel_idx), ptr(st.sel_cnt), None, None)
    assert rc == -2
