"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the
same seeded bf16 inputs.

Bars: page summaries bit-exact; selected-page sets exact except inside the 1e-5 relative
band around the oracle's k-th score; out within 1e-2 max-abs and 1e-3 mean-abs, lse within
1e-3 (attention is compared on the GPU's own selection, so a legal swap inside the band
cannot fail it); H2O increments within 1e-4 + 1e-3*value and summing to the group size.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39068_b200 import binding
from paper_2609_39068_b200 import workloads as wl
from helpers import check_selection, host_arrays

pytestmark = pytest.mark.gpu

OUT_MAX_ABS = 1e-2
OUT_MEAN_ABS = 1e-3
LSE_ABS = 1e-3


def run_gpu(w_cpu, accum=False, sink_pages=0, recent_pages=0):
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w, sink_pages=sink_pages, recent_pages=recent_pages)
    st.rebuild_meta()
    st.select()
    u = w.score_accum.clone() if accum else None
    st.decode(score_accum=u)
    torch.cuda.synchronize()
    assert st.status() == 0
    return w, st, u


def compare(w_cpu, st, rows=None, u_before=None, u_after=None, check_meta=True, sink_pages=0, recent_pages=0):
    a = host_arrays(w_cpu)
    rows = list(range(w_cpu.B)) if rows is None else list(rows)
    pt, sl, q = a["page_table"][rows], a["seq_lens"][rows], a["q"][rows]
    # --- summaries
    meta_gpu = wl.bf16_bits(st.meta)
    if check_meta:
        meta_ref = oracle.quest_meta(a["k"], pt, sl, first_tok=np.zeros(len(rows), np.int32), meta=meta_gpu)
        assert np.array_equal(meta_ref, meta_gpu), "page summaries differ"
    # --- selection
    S, P, present = oracle.quest_scores(q, meta_gpu, pt, sl)
    sel = st.sel_idx.cpu().numpy()[rows]
    cnt = st.sel_cnt.cpu().numpy()[rows]
    differing = check_selection(sel, cnt, P, present, w_cpu.budget, sink_pages=sink_pages,
                                recent_pages=recent_pages, seq_lens=sl)
    # A row may differ from the strict fp64 top-k only where the k-th and (k+1)-th scores are closer than
    # the fp32 scoring error (~3e-7 relative) - far rarer than a gap inside the 1e-5 band (a few percent
    # of the rows): more than 3 % of the rows differing means the scores are off, not tied.
    n_rows = len(rows) * w_cpu.H_kv
    assert differing <= max(1, (3 * n_rows + 99) // 100), \
        "%d of %d rows (%.1f %%) differ from the strict top-k inside the tie band" % (differing, n_rows, 100.0 * differing / n_rows)
    for r in range(len(rows)):
        for h in range(w_cpu.H_kv):
            row = sel[r, h, :cnt[r, h]]
            assert np.all(np.diff(row) > 0), "selection must be ascending"
    # --- attention on the GPU's selection
    u_ref = None
    if u_before is not None:
        u_ref = u_before.astype(np.float64).copy()
    out_ref, lse_ref = oracle.attend(q, a["k"], a["v"], pt, sl, sel, cnt, u_accum=u_ref)
    out = st.out.cpu().numpy()[rows].astype(np.float64)
    lse = st.lse.cpu().numpy()[rows].astype(np.float64)
    empty = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), empty)
    assert np.all(np.isfinite(out))
    err = np.abs(out - out_ref)
    assert err.max() <= OUT_MAX_ABS, err.max()
    assert err.mean() <= OUT_MEAN_ABS, err.mean()
    assert np.abs(lse[~empty] - lse_ref[~empty]).max(initial=0.0) <= LSE_ABS
    if u_before is not None:
        du_gpu = u_after.astype(np.float64) - u_before.astype(np.float64)
        du_ref = u_ref - u_before.astype(np.float64)
        assert np.all(np.abs(du_gpu - du_ref) <= 1e-4 + 1e-3 * du_ref + 2e-7 * np.abs(u_before))
        G = w_cpu.H_q // w_cpu.H_kv
        touched = du_ref != 0
        assert np.all(du_gpu[~touched] == 0)
    return dict(out_err=err.max(), differing=differing)


EDGE_CASES = {
    "len1":            dict(seq=[1], H_q=4, H_kv=1, D=128, budget=64),
    "len17_partial":   dict(seq=[17, 33, 16, 15], H_q=8, H_kv=2, D=128, budget=16, poison_tail=True),
    "k_ge_pages":      dict(seq=[100, 260, 40], H_q=8, H_kv=2, D=64, budget=16 * 32, poison_tail=True),
    "padding_slot":    dict(seq=[0, 300, 0, 77], H_q=8, H_kv=2, D=128, budget=64),
    "permuted":        dict(seq=[700, 1300, 257, 2049], H_q=8, H_kv=2, D=128, budget=256,
                            permute_pool=True, poison_tail=True, spare_pages=3),
    "aliased_prefix":  dict(seq=[900, 1100, 650], H_q=8, H_kv=2, D=128, budget=128,
                            permute_pool=True, shared_prefix_pages=20),
    "pruned":          dict(seq=[1500, 900, 333], H_q=8, H_kv=2, D=128, budget=128,
                            permute_pool=True, prune_fraction=0.3, poison_tail=True),
    "mostly_pruned":   dict(seq=[640, 320], H_q=4, H_kv=2, D=64, budget=128, prune_fraction=0.97),
    "outliers":        dict(seq=[3000, 1000], H_q=8, H_kv=2, D=128, budget=512, outliers=True),
    "many_requests":   dict(seq=list(range(5, 5 + 70 * 37, 37)), H_q=4, H_kv=2, D=64, budget=96,
                            permute_pool=True, poison_tail=True),
}


@pytest.mark.parametrize("name", sorted(EDGE_CASES))
def test_edge_cases(name):
    kw = dict(EDGE_CASES[name])
    seq = kw.pop("seq")
    w_cpu = wl.build(name, 800, 0, seq, kw.pop("H_q"), kw.pop("H_kv"), kw.pop("D"), kw.pop("budget"), "cpu", **kw)
    w, st, _ = run_gpu(w_cpu)
    compare(w_cpu, st)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
def test_every_group_size(D, G):
    w_cpu = wl.build("g", 810 + G, 0, [1234, 77, 600], 2 * G, 2, D, 160, "cpu", permute_pool=True,
                     poison_tail=True)
    w, st, _ = run_gpu(w_cpu)
    compare(w_cpu, st)


@pytest.mark.parametrize("sink,recent,budget", [(4, 16, 256), (0, 3, 64), (2, 0, 32), (6, 6, 16 * 200), (3, 5, 16)])
def test_forced_sink_and_recent_pages(sink, recent, budget):
    """Sink and recent pages are read in addition to the selected budget."""
    w_cpu = wl.build("forced", 825, 0, [2000, 50, 333, 16 * 4, 1], 8, 2, 128, budget, "cpu", permute_pool=True,
                     prune_fraction=0.15, poison_tail=True)
    w, st, _ = run_gpu(w_cpu, sink_pages=sink, recent_pages=recent)
    compare(w_cpu, st, sink_pages=sink, recent_pages=recent)
    # and the result is what the oracle selects, page for page, when no score is inside the band
    a = host_arrays(w_cpu)
    ref = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget,
                             meta=wl.bf16_bits(st.meta), sink_pages=sink, recent_pages=recent)
    assert np.array_equal(ref["sel_cnt"], st.sel_cnt.cpu().numpy())


def test_all_pages_pruned_gives_empty_result():
    w_cpu = wl.build("gone", 820, 0, [200, 90], 8, 2, 128, 64, "cpu")
    w_cpu.page_table[0, :] = -1
    w, st, _ = run_gpu(w_cpu)
    assert st.sel_cnt.cpu()[0].tolist() == [0, 0]
    assert torch.all(st.out[0] == 0) and torch.all(torch.isneginf(st.lse[0]))
    compare(w_cpu, st)


def test_budget_covering_everything_is_dense_attention():
    """Selected attention with every page selected must equal dense attention (torch SDPA, fp64)."""
    w_cpu = wl.build("dense", 830, 0, [777, 1500], 8, 2, 128, 16 * 128, "cpu", permute_pool=True)
    w, st, _ = run_gpu(w_cpu)
    a = host_arrays(w_cpu)
    from helpers import bits_to_f64, tokens_of_request
    K, V, Q = bits_to_f64(a["k"]), bits_to_f64(a["v"]), bits_to_f64(a["q"])
    for r in range(w_cpu.B):
        toks = tokens_of_request(a["page_table"][r], a["seq_lens"][r], 16)
        for h in range(w_cpu.H_kv):
            Kd = torch.from_numpy(np.stack([K[pid, h, t] for (_, t, pid) in toks]))[None, None]
            Vd = torch.from_numpy(np.stack([V[pid, h, t] for (_, t, pid) in toks]))[None, None]
            for g in range(4):
                head = h * 4 + g
                qq = torch.from_numpy(Q[r, head])[None, None, None]
                o = torch.nn.functional.scaled_dot_product_attention(qq, Kd, Vd)[0, 0, 0].numpy()
                assert np.abs(st.out[r, head].cpu().numpy() - o).max() <= OUT_MAX_ABS


def test_incremental_summary_update_matches_rebuild():
    """Append one token per request: updating only the newest page equals a rebuild."""
    w_cpu = wl.build("inc", 840, 0, [161, 320, 49, 16], 8, 2, 128, 64, "cpu", permute_pool=True)
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w)
    short = (w.seq_lens - 1).contiguous()
    ft = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    binding.se_meta_update(st.p, w.k_cache, w.page_table, short, st.meta, first_tok=ft)
    before = st.meta.clone()
    st.update_meta()                                   # only the page of the newest token
    inc = st.meta.clone()
    st.meta.zero_()
    st.rebuild_meta()
    torch.cuda.synchronize()
    assert torch.equal(inc.view(torch.int16), st.meta.view(torch.int16))
    assert not torch.equal(before.view(torch.int16), inc.view(torch.int16))
    # a rebuild from a given token on touches only pages from there
    st.meta.zero_()
    ft2 = torch.full((w.B,), 32, dtype=torch.int32, device="cuda")
    binding.se_meta_update(st.p, w.k_cache, w.page_table, w.seq_lens, st.meta, first_tok=ft2)
    torch.cuda.synchronize()
    pt = w.page_table.cpu()
    for r in range(w.B):
        n_r = (int(w.seq_lens[r]) + 15) // 16
        for b in range(n_r):
            touched = bool(st.meta[pt[r, b]].view(torch.int16).ne(0).any())
            assert touched == (b >= 2), (r, b)


@pytest.mark.parametrize("D,G", [(128, 4), (64, 2), (128, 7)])
def test_fused_summary_update_equals_separate_calls(D, G):
    """se_page_select_fused = se_meta_update (newest page) + se_page_select, bit for bit."""
    w_cpu = wl.build("fused", 845, 0, [161, 320, 49, 16, 1, 0, 2000], 2 * G, 2, D, 96, "cpu",
                     permute_pool=True, prune_fraction=0.1, poison_tail=True)
    w = w_cpu.to("cuda")
    short = (w.seq_lens - 1).clamp(min=0).contiguous()
    ft = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    states = []
    for fused in (False, True):
        st = binding.DecodeState(w)
        binding.se_meta_update(st.p, w.k_cache, w.page_table, short, st.meta, first_tok=ft)   # stale summaries
        if fused:
            st.select_fused()
        else:
            st.update_meta()
            st.select()
        st.decode()
        torch.cuda.synchronize()
        assert st.status() == 0
        states.append(st)
    a, b = states
    assert torch.equal(a.meta.view(torch.int16), b.meta.view(torch.int16))
    assert torch.equal(a.sel_idx, b.sel_idx) and torch.equal(a.sel_cnt, b.sel_cnt)
    assert torch.equal(a.out, b.out) and torch.equal(a.lse, b.lse)
    compare(w_cpu, b)


def test_summary_signed_zero_and_masking():
    w_cpu = wl.build("zero", 850, 0, [20], 2, 1, 64, 32, "cpu", poison_tail=True)
    w_cpu.k_cache[0, 0, 0, 0] = 0.0
    w_cpu.k_cache[0, 0, 1:, 0] = -0.0
    w_cpu.k_cache[0, 0, 0, 1] = -0.0
    w_cpu.k_cache[0, 0, 1:, 1] = 0.0
    w, st, _ = run_gpu(w_cpu)
    compare(w_cpu, st)
    bits = wl.bf16_bits(st.meta)
    assert bits[0, 0, 0, 0] == 0x8000 and bits[0, 0, 1, 0] == 0x0000
    assert bits[0, 0, 0, 1] == 0x8000 and bits[0, 0, 1, 1] == 0x0000


def test_ties_go_to_the_lower_page_and_inputs_are_not_written():
    """Identical pages score identically: the lower logical pages must win, and select/decode
    must leave q, K, V, summaries and the page table untouched."""
    w_cpu = wl.build("ties", 860, 0, [16 * 40], 4, 1, 128, 16 * 8, "cpu")
    w_cpu.k_cache[1:] = w_cpu.k_cache[0]
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w)
    st.rebuild_meta()
    torch.cuda.synchronize()
    snap = [t.clone() for t in (w.q, w.k_cache, w.v_cache, st.meta, w.page_table, w.seq_lens)]
    st.select()
    st.decode()
    torch.cuda.synchronize()
    assert st.sel_idx.cpu()[0, 0].tolist() == list(range(8))
    for s, t in zip(snap, (w.q, w.k_cache, w.v_cache, st.meta, w.page_table, w.seq_lens)):
        assert torch.equal(s.view(torch.uint8), t.view(torch.uint8))
    compare(w_cpu, st)


def test_two_runs_are_bit_identical_and_split_invariant():
    w_cpu = wl.build("det", 870, 0, [5000, 3000, 9000], 8, 2, 128, 1024, "cpu", permute_pool=True)
    w, st, _ = run_gpu(w_cpu)
    o1, l1, s1 = st.out.clone(), st.lse.clone(), st.sel_idx.clone()
    st.out.fill_(float("nan"))
    st.select()
    st.decode()
    torch.cuda.synchronize()
    assert torch.equal(o1, st.out) and torch.equal(l1, st.lse) and torch.equal(s1, st.sel_idx)
    # a larger k_max changes how the selected pages are split over warps, not the result
    st2 = binding.DecodeState(w, k_max=200)
    st2.rebuild_meta()
    st2.select()
    st2.decode()
    torch.cuda.synchronize()
    assert torch.equal(st2.sel_idx[:, :, :64], s1)
    assert (st2.out - o1).abs().max().item() <= 1e-5
    assert (st2.lse - l1).abs().max().item() <= 1e-5


def test_split_and_combine_calls_equal_the_single_call():
    w_cpu = wl.build("two", 875, 0, [5000, 300, 9000], 8, 2, 128, 1024, "cpu", permute_pool=True,
                     with_score_accum=True)
    w, st, u = run_gpu(w_cpu, accum=True)
    o1, l1 = st.out.clone(), st.lse.clone()
    st.out.fill_(float("nan"))
    st.lse.fill_(float("nan"))
    u2 = w.score_accum.clone()
    st.decode(u2, entry="se_sparse_decode_splits")
    st.decode(u2, entry="se_combine")
    torch.cuda.synchronize()
    assert torch.equal(o1, st.out) and torch.equal(l1, st.lse) and torch.equal(u, u2)


@pytest.mark.parametrize("fused", [False, True])
def test_dense_layer_mode_selects_every_present_page(fused):
    # budget >= context: nothing is scored, the selection is every present page in ascending order
    w_cpu = wl.build("dense", 877, 0, [700, 33, 16, 1, 1200], 8, 2, 128, 64, "cpu", permute_pool=True,
                     prune_fraction=0.3)
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w, k_max=w.max_pages)
    st.rebuild_meta()
    meta_full = st.meta.clone()
    if fused:
        st.meta.zero_()
        st.select_fused(budget=16 * w.max_pages)
    else:
        st.select(budget=16 * w.max_pages)
    torch.cuda.synchronize()
    a = host_arrays(w_cpu)
    sel, cnt = st.sel_idx.cpu().numpy(), st.sel_cnt.cpu().numpy()
    for r in range(w.B):
        n = (int(a["seq_lens"][r]) + 15) // 16
        want = [b for b in range(n) if a["page_table"][r, b] >= 0]
        for h in range(w.H_kv):
            assert cnt[r, h] == len(want) and sel[r, h, :len(want)].tolist() == want
            assert np.all(sel[r, h, len(want):] == -1)
    P = np.zeros((w.B, w.H_kv, w.max_pages))
    present = a["page_table"] >= 0
    for r in range(w.B):
        present[r, (int(a["seq_lens"][r]) + 15) // 16:] = False
    ref_idx, ref_cnt, _ = oracle.topk_pages(P, present, 16 * w.max_pages, k_max=w.max_pages)
    assert np.array_equal(ref_idx, sel) and np.array_equal(ref_cnt, cnt)
    if fused:       # the newest page's summary was still refreshed
        for r in range(w.B):
            pid = int(a["page_table"][r, (int(a["seq_lens"][r]) - 1) // 16])
            assert torch.equal(st.meta[pid], meta_full[pid])
    st.decode()
    torch.cuda.synchronize()
    assert st.status() == 0


def test_nan_in_slots_past_the_length_does_not_leak():
    # slots past a request's length are never initialised by an engine: NaN there must not matter
    w_cpu = wl.build("nan", 876, 0, [37, 16, 1, 250], 8, 2, 128, 64, "cpu", permute_pool=True,
                     with_score_accum=True)
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for r in range(w_cpu.B):
        L = int(w_cpu.seq_lens[r])
        if L % 16:
            pid = int(w_cpu.page_table[r, (L - 1) // 16])
            w_cpu.k_cache[pid, :, L % 16:, :] = nan
            w_cpu.v_cache[pid, :, L % 16:, :] = nan
    w, st, u = run_gpu(w_cpu, accum=True)
    assert torch.isfinite(st.out).all() and torch.isfinite(st.lse).all() and torch.isfinite(u).all()
    finite = w_cpu
    finite.k_cache = torch.nan_to_num(w_cpu.k_cache.float(), nan=0.0).to(torch.bfloat16)
    finite.v_cache = torch.nan_to_num(w_cpu.v_cache.float(), nan=0.0).to(torch.bfloat16)
    compare(finite, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy())


def test_score_and_topk_calls_equal_the_single_call():
    w_cpu = wl.build("two", 879, 0, [5000, 300, 9000], 8, 2, 128, 1024, "cpu", permute_pool=True)
    w, st, _ = run_gpu(w_cpu)
    s1, c1 = st.sel_idx.clone(), st.sel_cnt.clone()
    st.sel_idx.fill_(-5)
    st.sel_cnt.fill_(-5)
    st.select(entry="se_page_select_scores")
    torch.cuda.synchronize()
    assert int(st.sel_cnt[0, 0]) == -5            # the scoring half writes no selection
    st.select(entry="se_page_select_topk")
    torch.cuda.synchronize()
    assert torch.equal(s1, st.sel_idx) and torch.equal(c1, st.sel_cnt) and st.status() == 0


def test_h2o_accumulation_small():
    w_cpu = wl.build("h2o", 880, 0, [700, 1300, 90], 8, 2, 128, 256, "cpu", permute_pool=True,
                     with_score_accum=True, poison_tail=True)
    w, st, u = run_gpu(w_cpu, accum=True)
    res = compare(w_cpu, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy())
    # mass conservation: every (request, kv-head) adds exactly G
    du = (u - w.score_accum).double()
    assert abs(du.sum().item() - w_cpu.B * w_cpu.H_q) <= 1e-3 * w_cpu.B * w_cpu.H_q
    # a second step adds the same amount again
    st.decode(score_accum=u)
    torch.cuda.synchronize()
    du2 = (u - w.score_accum).double()
    assert torch.allclose(du2, 2 * du, rtol=1e-4, atol=1e-5)


def test_bad_selection_sets_status_and_is_skipped():
    w_cpu = wl.build("bad", 890, 0, [400, 400], 8, 2, 128, 64, "cpu")
    w, st, _ = run_gpu(w_cpu)
    good = st.out.clone()
    st.sel_idx[0, 0, 1] = 10_000                      # outside the request
    st.decode()
    torch.cuda.synchronize()
    assert st.status() & binding.SE_DEV_BAD_SELECTION
    assert torch.all(torch.isfinite(st.out))
    assert torch.equal(good[1], st.out[1])
    assert st.status() == 0                            # reading the status clears it


def _score_magnitude(a, meta_bits, r, h, G, n_r):
    """sm_scale * max over the group's heads of sum_c |q_c| * max(|min_c|, |max_c|) per page of (r, h):
    the size of the terms the score sums, which is what its fp32 rounding error scales with."""
    from helpers import bits_to_f64
    pt = a["page_table"][r, :n_r]
    pid = np.where(pt >= 0, pt, 0)
    m = bits_to_f64(meta_bits[pid, h])                        # [n_r, 2, D]
    big = np.maximum(np.abs(m[:, 0]), np.abs(m[:, 1]))         # [n_r, D]
    qa = np.abs(bits_to_f64(a["q"][r, h * G:(h + 1) * G]))     # [G, D]
    return (qa @ big.T).max(axis=0) / np.sqrt(qa.shape[1])


def _check_scores(w_cpu, st, a):
    got = binding.page_scores_view(st.p, st.workspace).cpu().numpy().astype(np.float64)
    meta_bits = wl.bf16_bits(st.meta)
    S, P, present = oracle.quest_scores(a["q"], meta_bits, a["page_table"], a["seq_lens"])
    G = w_cpu.H_q // w_cpu.H_kv
    n_checked, worst = 0, 0.0
    for r in range(w_cpu.B):
        n_r = (int(a["seq_lens"][r]) + 15) // 16
        for h in range(w_cpu.H_kv):
            row, ref, pres = got[r, h, :n_r], P[r, h, :n_r], present[r, :n_r]
            assert np.all(np.isneginf(row[~pres])), "absent pages must score -inf"
            mag = _score_magnitude(a, meta_bits, r, h, G, n_r)
            assert np.all(mag[pres] >= np.abs(ref[pres]) * (1 - 1e-12))
            rel = np.abs(row[pres] - ref[pres]) / mag[pres]
            worst = max(worst, float(rel.max(initial=0.0)))
            n_checked += int(pres.sum())
    assert worst <= 2e-6, worst
    return n_checked


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 4, 7, 8])
def test_page_scores_element_by_element(D, G):
    """The fp32 page scores themselves (not only which pages win) against the oracle's fp64 scores:
    every present page of every (request, kv-head) within 2e-6 of the size of the summed terms (<= 256 exact
    bf16 products accumulated in fp32 by the tensor cores), -inf on absent pages.  Pruned pages, partial last pages, an empty
    slot and outlier channels are in the mix."""
    w_cpu = wl.build("scores", 815 + G, 0, [1234, 77, 600, 0, 16, 4000], 2 * G, 2, D, 160, "cpu", permute_pool=True,
                     prune_fraction=0.2, poison_tail=True, outliers=True)
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.select(entry="se_page_select_scores")
    torch.cuda.synchronize()
    assert st.status() == 0
    n_checked = _check_scores(w_cpu, st, host_arrays(w_cpu))
    assert n_checked > 300


def test_page_scores_of_config2_element_by_element():
    w_cpu = wl.config2("cpu")
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.select(entry="se_page_select_scores")
    torch.cuda.synchronize()
    assert _check_scores(w_cpu, st, host_arrays(w_cpu)) == 8 * 8 * 2048


PLAN_CASES = dict(EDGE_CASES)
PLAN_CASES.update({
    "forced":       dict(seq=[2000, 50, 333, 64, 1, 0], H_q=8, H_kv=2, D=128, budget=256, permute_pool=True,
                         prune_fraction=0.15, sink=4, recent=16),
    "forced_only":  dict(seq=[40, 100], H_q=4, H_kv=2, D=64, budget=16, sink=3, recent=5),
    "long_d64":     dict(seq=[131072, 5], H_q=8, H_kv=1, D=64, budget=16 * 300, permute_pool=True),
    "all_selected": dict(seq=[3000, 200], H_q=8, H_kv=2, D=128, budget=16 * 188),
    "max_sizes":    dict(seq=[131072], H_q=8, H_kv=1, D=128, budget=65536, permute_pool=True),
})


@pytest.mark.parametrize("name", sorted(PLAN_CASES))
def test_decode_step_equals_the_separate_calls(name):
    """se_decode_step (scores -> top-k inside the attention kernel's prologue, in-kernel merge) must
    return what se_meta_update + se_page_select + se_sparse_decode return: summaries and selection bit for
    bit, out / lse bit for bit too (same pages, same split geometry), on a first and a second call."""
    kw = dict(PLAN_CASES[name])
    seq, sink, recent = kw.pop("seq"), kw.pop("sink", 0), kw.pop("recent", 0)
    accum = "shared_prefix_pages" not in kw           # the H2O epilogue does not allow aliased pages
    w = wl.build(name, 800, 0, seq, kw.pop("H_q"), kw.pop("H_kv"), kw.pop("D"), kw.pop("budget"), "cuda",
                 with_score_accum=True, **kw)
    short = (w.seq_lens - 1).clamp(min=0).contiguous()
    ft = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    res = []
    for fused in (False, True, True):
        st = binding.DecodeState(w, sink_pages=sink, recent_pages=recent)
        binding.se_meta_update(st.p, w.k_cache, w.page_table, short, st.meta, first_tok=ft)   # stale newest page
        u = w.score_accum.clone()
        st.step(score_accum=u if accum else None, fused=fused)
        torch.cuda.synchronize()
        assert st.status() == 0
        # the fp32 page scores left in the workspace (whichever kernel wrote them), up to each request's last page
        sc = binding.page_scores_view(st.p, st.workspace).clone()
        for r in range(w.B):
            sc[r, :, (int(w.seq_lens[r]) + 15) // 16:] = 0
        if w.budget // 16 >= w.max_pages:
            sc.zero_()                        # dense-layer mode: nothing is scored
        res.append((st.meta.view(torch.int16).clone(), st.sel_idx.clone(), st.sel_cnt.clone(), st.out.clone(),
                    st.lse.clone(), u, sc.view(torch.int32)))
    for other in res[1:]:
        for x, y in zip(res[0], other):
            assert torch.equal(x, y)


def test_ties_with_selection_inside_the_attention_kernel():
    w_cpu = wl.build("ties", 860, 0, [16 * 40, 16 * 700], 4, 1, 128, 16 * 8, "cpu")
    w_cpu.k_cache[1:] = w_cpu.k_cache[0]
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.step()
    torch.cuda.synchronize()
    assert st.sel_idx.cpu()[0, 0].tolist() == list(range(8)) and st.sel_idx.cpu()[1, 0].tolist() == list(range(8))
    compare(w_cpu, st)


@pytest.mark.parametrize("pairs", [2, 40, 148, 200, 400, 592, 700])
def test_every_launch_plan_against_the_oracle(pairs):
    """The attention step has four geometries, picked from the number of (request, kv-head) pairs: CTA
    units in a cluster (<= 148 pairs), warp units with splits and the merge kernel (< 296), two warps per
    pair (<= 592), one warp per pair (more).  Each one against the oracle, with and without the H2O
    epilogue."""
    H_kv = 2 if pairs % 2 == 0 else 1
    B = pairs // H_kv
    rng = np.random.default_rng(pairs)
    seq = [int(x) for x in rng.integers(1, 2500, size=B)]
    seq[0] = 0
    for accum in (False, True):
        w_cpu = wl.build("plan%d" % pairs, 897, 0, seq, 4 * H_kv, H_kv, 128, 320, "cpu", permute_pool=True,
                         prune_fraction=0.1, with_score_accum=True, poison_tail=True)
        w = w_cpu.to("cuda")
        st = binding.DecodeState(w)
        st.rebuild_meta()
        u = w.score_accum.clone() if accum else None
        st.step(score_accum=u)
        torch.cuda.synchronize()
        assert st.status() == 0
        if accum:
            compare(w_cpu, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy())
        else:
            compare(w_cpu, st)


def test_maximum_batch_of_short_requests():
    """The largest batch the library takes (8192 requests: the scoring kernel's per-request tables fill
    a third of its shared memory, so it runs with one CTA per SM), one to five pages each."""
    rng = np.random.default_rng(8192)
    seq = [int(x) for x in rng.integers(1, 80, size=8192)]
    seq[17] = 0
    w_cpu = wl.build("maxbatch", 899, 0, seq, 2, 1, 64, 32, "cpu", permute_pool=True)
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.step()
    torch.cuda.synchronize()
    assert st.status() == 0
    compare(w_cpu, st)


def _run_shard(w, accum):
    st = binding.DecodeState(w)
    short = (w.seq_lens - 1).clamp(min=0).contiguous()
    ft = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    binding.se_meta_update(st.p, w.k_cache, w.page_table, short, st.meta, first_tok=ft)
    u = w.score_accum.clone() if accum else None
    st.step(score_accum=u)
    torch.cuda.synchronize()
    assert st.status() == 0
    return st, u


@pytest.mark.parametrize("many_pairs", [True, False])
def test_kv_head_shards_reproduce_the_unsharded_step(many_pairs):
    """Tensor-parallel sharding by kv-head needs no exchange: the CUDA step run on the two shards of
    wl.shard_kv_heads, concatenated, is the unsharded CUDA step.  With enough pairs that neither run splits
    a pair (many_pairs) every output is bit-identical; with few pairs the split-K geometry differs
    between the shapes, so out/lse/score_accum agree to fp32 rounding and the rest bit for bit."""
    if many_pairs:
        seq = [300 + 23 * i for i in range(160)]            # 160 requests x 8 kv-heads: 640 pairs per shard (one warp per pair in both runs)
    else:
        seq = [5000, 3000, 9000, 17]
    w = wl.build("tp", 895, 0, seq, 16, 8, 128, 256, "cpu", permute_pool=True, prune_fraction=0.1,
                 with_score_accum=True, poison_tail=True).to("cuda")
    full, u_full = _run_shard(w, True)
    if many_pairs:
        assert binding.se_decode_num_splits(full.p) == 1
    parts = [_run_shard(wl.shard_kv_heads(w, r, 2), True) for r in range(2)]
    if many_pairs:
        assert all(binding.se_decode_num_splits(st.p) == 1 for st, _ in parts)
    cat = lambda f, dim: torch.cat([f(st, u) for st, u in parts], dim=dim)
    assert torch.equal(cat(lambda st, u: st.meta.view(torch.int16), 1), full.meta.view(torch.int16))
    assert torch.equal(cat(lambda st, u: st.sel_idx, 1), full.sel_idx)
    assert torch.equal(cat(lambda st, u: st.sel_cnt, 1), full.sel_cnt)
    out, lse, acc = cat(lambda st, u: st.out, 1), cat(lambda st, u: st.lse, 1), cat(lambda st, u: u, 1)
    if many_pairs:
        assert torch.equal(out, full.out) and torch.equal(lse, full.lse) and torch.equal(acc, u_full)
    else:
        assert (out - full.out).abs().max().item() <= 1e-5 and (lse - full.lse).abs().max().item() <= 1e-5
        assert (acc - u_full).abs().max().item() <= 1e-5


# ---------------------------------------------------------------- the named configurations

def test_maximum_sizes_one_request():
    # the limits of the build at once: 131072 tokens (8192 pages), k_max = 4096 selected pages, G = 8
    w = wl.build("max", 878, 0, [131072], 8, 1, 128, 65536, "cuda", permute_pool=True)
    w_cpu = w.to("cpu")
    st = binding.DecodeState(w)
    assert st.k_max == 4096 and w.max_pages == 8192
    st.rebuild_meta()
    st.step()
    torch.cuda.synchronize()
    assert st.status() == 0
    compare(w_cpu, st)


def test_config1_tiny():
    w_cpu = wl.config1("cpu")
    w, st, _ = run_gpu(w_cpu)
    compare(w_cpu, st)


def test_config2_llama8b_layer():
    w_cpu = wl.config2("cpu")
    w, st, _ = run_gpu(w_cpu)
    compare(w_cpu, st)


def _gpu_built(cfg_fn, **kw):
    """Full-size workload generated on the GPU; the host copy for the oracle shares its bits."""
    w = cfg_fn("cuda", **kw)
    return w, w.to("cpu")


def test_config3_full_size_all_requests():
    w, w_cpu = _gpu_built(wl.config3)
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.step()
    torch.cuda.synchronize()
    assert st.status() == 0
    compare(w_cpu, st)                       # every one of the 64 requests
    _check_scores(w_cpu, st, host_arrays(w_cpu))


def test_config4_long_context_with_h2o():
    w, w_cpu = _gpu_built(wl.config4)
    st = binding.DecodeState(w)
    st.rebuild_meta()
    u = w.score_accum.clone()
    st.step(score_accum=u)
    torch.cuda.synchronize()
    assert st.status() == 0
    compare(w_cpu, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy())
    du = (u - w.score_accum).double()
    assert abs(du.sum().item() - w.B * w.H_q) <= 1e-3 * w.B * w.H_q


@pytest.mark.parametrize("layer", [0, 13, 27])
def test_config5_one_layer_all_requests(layer):
    torch.cuda.empty_cache()
    w, w_cpu = _gpu_built(wl.config5, layer=layer)
    st = binding.DecodeState(w)
    st.rebuild_meta()
    st.step()
    torch.cuda.synchronize()
    assert st.status() == 0
    compare(w_cpu, st)                       # every one of the 128 requests
    _check_scores(w_cpu, st, host_arrays(w_cpu))


def test_config5_28_layer_graph_replay_matches_oracle():
    """The step the benchmark times - 28 layers captured in one CUDA graph, all layers sharing one
    workspace - is the checked computation: after two replays the summaries, selections and outputs of
    layers 0, 13 and 27 are compared with the oracle for every request, and the second replay must
    reproduce the first bit for bit."""
    torch.cuda.empty_cache()
    n_layers, check = 28, (0, 13, 27)
    layers = [wl.config5("cuda", layer=l) for l in range(n_layers)]
    for w in layers[1:]:                     # the block table is per request, shared by all layers
        w.page_table, w.seq_lens = layers[0].page_table, layers[0].seq_lens
    states = [binding.DecodeState(layers[0])]
    for w in layers[1:]:
        states.append(binding.DecodeState(w, workspace=states[0].workspace))
    # stale summaries for each request's newest page: the fused step has to refresh them
    short = (layers[0].seq_lens - 1).contiguous()
    ft = torch.zeros(layers[0].B, dtype=torch.int32, device="cuda")
    for st in states:
        binding.se_meta_update(st.p, st.w.k_cache, st.w.page_table, short, st.meta, first_tok=ft)

    def step():
        for st in states:
            st.step()

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for st in states:
        st.out.fill_(float("nan")); st.lse.fill_(float("nan")); st.sel_idx.fill_(-7); st.sel_cnt.fill_(-7)
    graph.replay()
    torch.cuda.synchronize()
    first = {l: (states[l].out.clone(), states[l].lse.clone(), states[l].sel_idx.clone()) for l in check}
    for st in states:
        st.out.fill_(float("nan")); st.lse.fill_(float("nan")); st.sel_idx.fill_(-7); st.sel_cnt.fill_(-7)
    graph.replay()
    torch.cuda.synchronize()
    assert states[0].status() == 0
    for st in states:
        assert torch.isfinite(st.out).all() and int(st.sel_cnt.min()) >= 0
    for l in check:
        o, ls, si = first[l]
        assert torch.equal(o, states[l].out) and torch.equal(ls, states[l].lse) and torch.equal(si, states[l].sel_idx)
        compare(layers[l].to("cpu"), states[l])
    del graph


def test_config5_dense_first_layers_in_one_graph():
    """Per-layer policy of the paper's Quest settings: the first two layers attend everything (dense-layer
    mode: budget >= context), the others select under the budget - all captured in ONE graph with a
    shared workspace.  Small version of the config-5 recipe (16 requests, 6 layers)."""
    torch.cuda.empty_cache()
    n_layers, n_dense = 6, 2
    layers = [wl.config5("cuda", layer=l, B=16) for l in range(n_layers)]
    for w in layers[1:]:
        w.page_table, w.seq_lens = layers[0].page_table, layers[0].seq_lens
    mp = layers[0].max_pages
    big = binding.DecodeState(layers[0], k_max=mp)            # sized for the dense layers
    states = [big] + [binding.DecodeState(w, k_max=mp if l + 1 < n_dense else None, workspace=big.workspace)
                      for l, w in enumerate(layers[1:])]
    for st in states:
        st.rebuild_meta()

    def step():
        for l, st in enumerate(states):
            if l < n_dense:
                st.select_fused(budget=16 * mp)
                st.decode()
            else:
                st.step()

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for st in states:
        st.out.fill_(float("nan")); st.lse.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    assert big.status() == 0
    for l, st in enumerate(states):
        w_cpu = layers[l].to("cpu")
        if l < n_dense:
            w_cpu.budget = 16 * mp
        compare(w_cpu, st)
    del graph
