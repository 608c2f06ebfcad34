"""The bounded waits: a copy that never completes must end in SE_DEV_WAIT_TIMEOUT, not in a hang.

A second build of the library (``-DSE_TEST_SHORT_TX``) makes every batch of the scoring kernel announce
16 bytes more than its copies deliver, so each warp's first wait runs out after the limit (200 ms of
%globaltimer); the kernel sets the status bit, waits - bounded again - for what it still has in
flight, checks out of the work queue and returns.  Nothing faults and nothing spins forever.  The
workspace must be usable by the next call as it is."""
import ctypes
import time

import pytest
import torch

from paper_2609_39068_b200 import _build, binding
from paper_2609_39068_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_wait_that_never_completes_times_out_and_leaves_the_workspace_usable():
    w = wl.build("timeout", 995, 0, [700, 90, 2049], 8, 2, 128, 256, "cpu", permute_pool=True).to("cuda")
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.select()
    torch.cuda.synchronize()
    assert st.status() == 0
    good_idx, good_cnt = st.sel_idx.clone(), st.sel_cnt.clone()

    lib = ctypes.CDLL(_build.build_short_tx())
    ptr = lambda t: ctypes.c_void_p(t.data_ptr())
    lib.se_page_select.restype = ctypes.c_int
    t0 = time.perf_counter()
    rc = lib.se_page_select(ctypes.byref(st.p), ptr(w.q), ptr(st.meta), ptr(w.page_table), ptr(w.seq_lens),
                            ctypes.c_int32(w.budget), ptr(st.sel_idx), ptr(st.sel_cnt), ptr(st.workspace),
                            ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0
    torch.cuda.synchronize()                      # returns: the kernel gave up by itself
    elapsed = time.perf_counter() - t0
    assert 0.15 < elapsed < 5.0, elapsed          # one or two wait limits, not forever
    assert st.status() == binding.SE_DEV_WAIT_TIMEOUT
    assert st.status() == 0                       # reading the status cleared it

    # the next call on the same workspace, no re-initialisation: the work-queue counters were left at zero
    st.sel_idx.fill_(-7)
    st.sel_cnt.fill_(-7)
    st.select()
    torch.cuda.synchronize()
    assert st.status() == 0
    assert torch.equal(st.sel_idx, good_idx) and torch.equal(st.sel_cnt, good_cnt)
