"""GPU parity of the H2O retention / eviction calls against the CPU oracle, through the C ABI.
Retained positions, moved K/V rows and scores are integer / byte work: compared bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39068_b200 import binding, workloads as wl
from helpers import host_arrays

pytestmark = pytest.mark.gpu


def make(seed, seq, H_q=8, H_kv=2, D=128, levels=None, **kw):
    w = wl.build("h2o", 960 + seed, 0, list(seq), H_q, H_kv, D, 64, "cpu", with_score_accum=True, **kw)
    if levels:      # few distinct score values: crowded histogram bins and ties
        w.score_accum = torch.round(w.score_accum * levels) / levels
    return w


def gpu_retain(w, budget, recent):
    p = binding.make_params(w.B, w.H_q, w.H_kv, w.D, w.max_pages, w.num_phys_pages, 1)
    ws = binding.alloc_workspace(p, "cuda")
    keep_idx = torch.full((w.B, w.H_kv, budget), -9, dtype=torch.int32, device="cuda")
    keep_cnt = torch.full((w.B, w.H_kv), -9, dtype=torch.int32, device="cuda")
    binding.se_h2o_retain(p, w.score_accum, w.page_table, w.seq_lens, budget, recent, keep_idx, keep_cnt, ws)
    torch.cuda.synchronize()
    assert binding.se_last_device_status(ws) == 0
    return p, ws, keep_idx, keep_cnt


def check_retain(w_cpu, budget, recent, rows=None):
    w = w_cpu.to("cuda")
    u_before = w.score_accum.clone()
    p, ws, keep_idx, keep_cnt = gpu_retain(w, budget, recent)
    assert torch.equal(u_before, w.score_accum), "se_h2o_retain must not write the scores"
    a = host_arrays(w_cpu)
    rows = list(range(w_cpu.B)) if rows is None else list(rows)
    ref_idx, ref_cnt = oracle.h2o_retain(w_cpu.score_accum.numpy().astype(np.float64), a["page_table"][rows],
                                         a["seq_lens"][rows], budget, recent)
    assert np.array_equal(keep_cnt.cpu().numpy()[rows], ref_cnt)
    assert np.array_equal(keep_idx.cpu().numpy()[rows], ref_idx)
    return w, p, ws, keep_idx, keep_cnt


@pytest.mark.parametrize("budget,recent", [(32, 8), (32, 0), (32, 32), (32, 100), (16, 5), (300, 10), (1, 1), (1, 0)])
def test_retain_small(budget, recent):
    check_retain(make(1, (70, 33, 16, 1, 120, 257), permute_pool=True), budget, recent)


@pytest.mark.parametrize("levels", [1, 4, 64])
def test_retain_with_ties_and_crowded_bins(levels):
    check_retain(make(2, (5000, 4097, 300), levels=levels, permute_pool=True), 1024, 100)
    check_retain(make(2, (5000, 4097, 300), levels=levels, permute_pool=True), 4096, 819)


def test_retain_long_requests_and_pruned_pages():
    w = make(3, (20000, 9000, 4500), prune_fraction=0.2, permute_pool=True)
    check_retain(w, 4096, 2048)
    check_retain(w, 8192, 16)


def test_retain_all_scores_equal():
    w = make(4, (700, 64))
    w.score_accum = torch.full_like(w.score_accum, 0.25)
    check_retain(w, 256, 32)


@pytest.mark.parametrize("D,H_q,H_kv", [(128, 8, 2), (64, 4, 4)])
def test_compact_matches_oracle_and_preserves_attention(D, H_q, H_kv):
    w_cpu = make(5, (1300, 520, 40, 16), H_q=H_q, H_kv=H_kv, D=D, permute_pool=True)
    budget, recent = 512, 100
    w, p, ws, keep_idx, keep_cnt = check_retain(w_cpu, budget, recent)
    a = host_arrays(w_cpu)
    u64 = w_cpu.score_accum.numpy().astype(np.float64)
    k_ref, v_ref, u_ref, len_ref = oracle.h2o_compact(a["k"], a["v"], u64, a["page_table"],
                                                      keep_idx.cpu().numpy(), keep_cnt.cpu().numpy())
    new_lens = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    assert binding.se_last_device_status(ws) == 0
    assert np.array_equal(new_lens.cpu().numpy(), len_ref)
    assert np.array_equal(wl.bf16_bits(w.k_cache), k_ref)
    assert np.array_equal(wl.bf16_bits(w.v_cache), v_ref)
    assert np.array_equal(w.score_accum.cpu().numpy().astype(np.float64), u_ref)
    # dense decode over the compacted cache == oracle attention over the retained tokens of the old one
    w2 = wl.Workload(**{**w.__dict__, "seq_lens": new_lens, "budget": 16 * w.max_pages})
    st = binding.DecodeState(w2, k_max=w.max_pages)
    st.rebuild_meta()
    st.select()
    st.decode()
    torch.cuda.synchronize()
    assert st.status() == 0
    n_pages = (len_ref + 15) // 16
    sel = np.full((w.B, w.H_kv, w.max_pages), -1, np.int32)
    scnt = np.zeros((w.B, w.H_kv), np.int32)
    for r in range(w.B):
        sel[r, :, :n_pages[r]] = np.arange(n_pages[r])
        scnt[r, :] = n_pages[r]
    out, lse = oracle.attend(a["q"], k_ref, v_ref, a["page_table"], len_ref, sel, scnt)
    assert np.abs(st.out.cpu().numpy() - out).max() <= 1e-2
    assert np.abs(st.lse.cpu().numpy() - lse).max() <= 1e-3


def test_compact_twice_is_stable_and_bad_rows_are_reported():
    w_cpu = make(6, (300, 200))
    w, p, ws, keep_idx, keep_cnt = check_retain(w_cpu, 128, 16)
    new_lens = torch.zeros((w.B,), dtype=torch.int32, device="cuda")
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    k1 = w.k_cache.clone()
    # after the eviction the request is at its budget: nothing more to evict, compaction is the identity
    w.seq_lens = new_lens
    binding.se_h2o_retain(p, w.score_accum, w.page_table, w.seq_lens, 128, 16, keep_idx, keep_cnt, ws)
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    assert torch.equal(k1, w.k_cache) and new_lens.tolist() == [128, 128]
    assert keep_idx[0, 0].tolist() == list(range(128))
    # a source before its destination is skipped and flagged, nothing faults
    bad = keep_idx.clone()
    bad[0, 0, 100] = 3
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, bad, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    assert binding.se_last_device_status(ws) & binding.SE_DEV_BAD_SELECTION
    assert torch.equal(k1, w.k_cache)


def test_eviction_workload_full_size_sampled():
    # the periodic decode eviction of the paper's H2O settings: 4096-token budget, eviction every
    # 1024 steps (5120 cached tokens), recent ratio 0.2, 64 concurrent requests
    w_cpu = wl.h2o_evict_workload("cpu")
    rows = [0, 17, 63]
    w, p, ws, keep_idx, keep_cnt = check_retain(w_cpu, 4096, 819, rows=rows)
    sub = wl.sub_workload(w_cpu, rows)
    a = host_arrays(sub)
    ki, kc = keep_idx.cpu().numpy()[rows], keep_cnt.cpu().numpy()[rows]
    k_ref, v_ref, u_ref, len_ref = oracle.h2o_compact(a["k"], a["v"], sub.score_accum.numpy().astype(np.float64),
                                                      a["page_table"], ki, kc)
    new_lens = torch.zeros((w.B,), dtype=torch.int32, device="cuda")
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    assert binding.se_last_device_status(ws) == 0
    assert new_lens.tolist() == [4096] * w.B
    got = wl.sub_workload(w.to("cpu"), rows)
    assert np.array_equal(wl.bf16_bits(got.k_cache), k_ref)
    assert np.array_equal(wl.bf16_bits(got.v_cache), v_ref)
    assert np.array_equal(got.score_accum.numpy().astype(np.float64), u_ref)


def test_h2o_lifecycle_decode_evict_decode():
    """Scores accumulate during a dense decode step, the eviction keeps the heavy hitters and the recent
    window, and the next decode step runs on the compacted cache with the scores still aligned: every
    stage against the oracle doing the same."""
    w_cpu = wl.build("life", 966, 0, [400, 150, 64], 8, 2, 128, 64, "cpu", permute_pool=True, with_score_accum=True)
    w_cpu.score_accum.zero_()                       # scores start at zero
    w = w_cpu.to("cuda")
    a = host_arrays(w_cpu)
    n_pages = (a["seq_lens"] + 15) // 16
    sel = np.full((w.B, w.H_kv, w.max_pages), -1, np.int32)
    scnt = np.zeros((w.B, w.H_kv), np.int32)
    for r in range(w.B):
        sel[r, :, :n_pages[r]] = np.arange(n_pages[r])
        scnt[r, :] = n_pages[r]
    # step 1: full attention, scores accumulate
    st = binding.DecodeState(w, k_max=w.max_pages)
    st.sel_idx.copy_(torch.from_numpy(sel))
    st.sel_cnt.copy_(torch.from_numpy(scnt))
    st.decode(score_accum=w.score_accum)
    torch.cuda.synchronize()
    u_ref = np.zeros_like(w_cpu.score_accum.numpy(), dtype=np.float64)
    oracle.attend(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], sel, scnt, u_accum=u_ref)
    u_gpu = w.score_accum.cpu().numpy().astype(np.float64)
    assert np.abs(u_gpu - u_ref).max() <= 1e-4 + 1e-3 * np.abs(u_ref).max()
    # eviction on the GPU's own fp32 scores: bit-exact against the oracle fed with them
    budget, recent = 96, 16
    p, ws, keep_idx, keep_cnt = gpu_retain(w, budget, recent)
    ref_idx, ref_cnt = oracle.h2o_retain(u_gpu, a["page_table"], a["seq_lens"], budget, recent)
    assert np.array_equal(keep_idx.cpu().numpy(), ref_idx) and np.array_equal(keep_cnt.cpu().numpy(), ref_cnt)
    k2, v2, u2, len2 = oracle.h2o_compact(a["k"], a["v"], u_gpu, a["page_table"], ref_idx, ref_cnt)
    new_lens = torch.zeros((w.B,), dtype=torch.int32, device="cuda")
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    assert np.array_equal(new_lens.cpu().numpy(), len2) and np.array_equal(wl.bf16_bits(w.k_cache), k2)
    # step 2: the next decode step on the compacted cache keeps accumulating on the moved scores
    n2 = (len2 + 15) // 16
    sel2 = np.full_like(sel, -1)
    scnt2 = np.zeros_like(scnt)
    for r in range(w.B):
        sel2[r, :, :n2[r]] = np.arange(n2[r])
        scnt2[r, :] = n2[r]
    w2 = wl.Workload(**{**w.__dict__, "seq_lens": new_lens})
    st2 = binding.DecodeState(w2, k_max=w.max_pages)
    st2.sel_idx.copy_(torch.from_numpy(sel2))
    st2.sel_cnt.copy_(torch.from_numpy(scnt2))
    st2.decode(score_accum=w.score_accum)
    torch.cuda.synchronize()
    assert st2.status() == 0
    out_ref, lse_ref = oracle.attend(a["q"], k2, v2, a["page_table"], len2, sel2, scnt2, u_accum=u2)
    assert np.abs(st2.out.cpu().numpy() - out_ref).max() <= 1e-2
    assert np.abs(st2.lse.cpu().numpy() - lse_ref).max() <= 1e-3
    assert np.abs(w.score_accum.cpu().numpy().astype(np.float64) - u2).max() <= 1e-4 + 1e-3 * np.abs(u2).max()
