"""GPU parity of the selection-reuse path (observation layer scores, token selection, token-granular
attention) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39068_b200 import binding, workloads as wl
from helpers import host_arrays

pytestmark = pytest.mark.gpu

OUT_MAX_ABS, OUT_MEAN_ABS, LSE_ABS = 1e-2, 1e-3, 1e-3


def observe(w, recent=0, budget=None):
    """Dense observation layer on the GPU: returns (state, tok_keys)."""
    st = binding.DecodeState(w, k_max=w.max_pages)
    st.w = wl.Workload(**{**w.__dict__, "budget": 16 * w.max_pages})
    st.rebuild_meta()
    st.select()                                    # budget >= context: every present page
    keys = torch.full((w.B, 16 * w.max_pages), 0x55, dtype=torch.int32, device="cuda")
    binding.se_observe_decode(st.p, w.q, w.k_cache, w.v_cache, w.page_table, w.seq_lens, st.sel_idx, st.sel_cnt,
                              st.out, st.lse, keys, st.workspace)
    torch.cuda.synchronize()
    assert st.status() == 0
    return st, keys


def check_scores(w_cpu, keys, rows=None):
    a = host_arrays(w_cpu)
    rows = list(range(w_cpu.B)) if rows is None else rows
    s_ref, present = oracle.token_scores(a["q"][rows], a["k"], a["page_table"][rows], a["seq_lens"][rows])
    s_gpu, att = binding.keys_to_scores(keys)
    s_gpu, att = s_gpu.cpu().numpy()[rows], att.cpu().numpy()[rows]
    assert np.array_equal(att, present)
    err = np.abs(s_gpu.astype(np.float64) - s_ref)[present]
    assert err.max() <= 1e-4 * max(1.0, np.abs(s_ref[present]).max()), err.max()
    return s_ref, present, s_gpu


def select(st, keys, w, budget, recent):
    n_out = budget + recent
    tok_idx = torch.full((w.B, n_out), -9, dtype=torch.int32, device="cuda")
    tok_cnt = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
    binding.se_token_select(st.p, keys, w.seq_lens, budget, recent, tok_idx, tok_cnt, st.workspace)
    torch.cuda.synchronize()
    assert st.status() == 0
    return tok_idx, tok_cnt


def check_select(w_cpu, s_ref, present, s_gpu, tok_idx, tok_cnt, budget, recent, rows=None):
    a = host_arrays(w_cpu)
    rows = list(range(w_cpu.B)) if rows is None else rows
    sl = a["seq_lens"][rows]
    got_idx, got_cnt = tok_idx.cpu().numpy()[rows], tok_cnt.cpu().numpy()[rows]
    # the decision is taken on the GPU's own fp32 scores: the oracle fed with them agrees exactly
    ref_idx, ref_cnt, _ = oracle.token_topk(s_gpu.astype(np.float64), present, sl, budget, recent)
    assert np.array_equal(got_cnt, ref_cnt) and np.array_equal(got_idx, ref_idx)
    # against the oracle's fp64 scores: everything clearly above the threshold is in, nothing clearly below
    _, _, theta = oracle.token_topk(s_ref, present, sl, budget, recent)
    for i in range(len(rows)):
        L = int(sl[i])
        chosen = set(got_idx[i, :got_cnt[i]].tolist())
        if np.isnan(theta[i]):
            continue
        eps = 1e-4 * max(1.0, abs(theta[i]))
        comp = [j for j in range(L - recent) if present[i, j]] if L > recent else []
        assert all(j in chosen for j in comp if s_ref[i, j] > theta[i] + eps)
        assert not any(j in chosen for j in comp if s_ref[i, j] < theta[i] - eps)


def token_decode(w, p, ws, tok_idx, tok_cnt):
    out = torch.full((w.B, w.H_q, w.D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((w.B, w.H_q), float("nan"), dtype=torch.float32, device="cuda")
    binding.se_token_decode(p, w.q, w.k_cache, w.v_cache, w.page_table, w.seq_lens, tok_idx, tok_cnt, out, lse, ws)
    torch.cuda.synchronize()
    return out, lse


def check_attend(w_cpu, tok_idx, tok_cnt, out, lse, rows=None):
    a = host_arrays(w_cpu)
    rows = list(range(w_cpu.B)) if rows is None else rows
    o_ref, l_ref = oracle.token_attend(a["q"][rows], a["k"], a["v"], a["page_table"][rows], a["seq_lens"][rows],
                                       tok_idx.cpu().numpy()[rows], tok_cnt.cpu().numpy()[rows])
    o, l = out.cpu().numpy()[rows], lse.cpu().numpy()[rows]
    assert np.abs(o - o_ref).max() <= OUT_MAX_ABS and np.abs(o - o_ref).mean() <= OUT_MEAN_ABS
    fin = np.isfinite(l_ref)
    assert np.array_equal(np.isneginf(l), np.isneginf(l_ref))
    assert np.abs(l[fin] - l_ref[fin]).max(initial=0.0) <= LSE_ABS


# (one to sixteen kv-heads and both head sizes: the kernel's work units are (request, kv-head, token chunk))
@pytest.mark.parametrize("D,H_q,H_kv", [(128, 8, 2), (64, 4, 4), (128, 7, 1), (128, 16, 16), (64, 8, 8)])
@pytest.mark.parametrize("prune", [0.0, 0.3])
def test_observe_select_reuse_small(D, H_q, H_kv, prune):
    w_cpu = wl.build("tok", 980, 0, [700, 300, 17, 1, 1200], H_q, H_kv, D, 64, "cpu", permute_pool=True,
                     prune_fraction=prune, poison_tail=True)
    w = w_cpu.to("cuda")
    st, keys = observe(w)
    # the observation output does not change the attention result
    st2 = binding.DecodeState(w, k_max=w.max_pages)
    st2.w, st2.sel_idx, st2.sel_cnt = st.w, st.sel_idx, st.sel_cnt
    st2.decode()
    torch.cuda.synchronize()
    # (an observation layer runs on warp units, the plain call may run on CTA units: same pages, another
    # split geometry, hence fp32 rounding)
    assert (st.out - st2.out).abs().max().item() <= 1e-5 and (st.lse - st2.lse).abs().max().item() <= 1e-5
    s_ref, present, s_gpu = check_scores(w_cpu, keys)
    for budget, recent in [(64, 8), (200, 0), (16, 40), (2000, 4), (0, 8)]:
        tok_idx, tok_cnt = select(st, keys, w, budget, recent)
        check_select(w_cpu, s_ref, present, s_gpu, tok_idx, tok_cnt, budget, recent)
        # two sparse layers reuse the set on their own caches
        for layer in (1, 2):
            wl_cpu = wl.build("tok", 980, layer, [700, 300, 17, 1, 1200], H_q, H_kv, D, 64, "cpu",
                              permute_pool=True, prune_fraction=prune, poison_tail=True)
            assert torch.equal(wl_cpu.page_table, w_cpu.page_table)
            wlg = wl_cpu.to("cuda")
            p = binding.make_params(w.B, H_q, H_kv, D, w.max_pages, w.num_phys_pages, (budget + recent + 15) // 16)
            ws = binding.alloc_workspace(p, "cuda")
            out, lse = token_decode(wlg, p, ws, tok_idx, tok_cnt)
            assert binding.se_last_device_status(ws) == 0
            check_attend(wl_cpu, tok_idx, tok_cnt, out, lse)


def test_token_decode_many_pairs_no_split_and_arbitrary_sets():
    # 40 requests x 8 heads: the plan does not split; hand-made sets with repeats of pages, ragged counts
    seq = [200 + 37 * i for i in range(40)]
    w_cpu = wl.build("tok", 981, 0, seq, 32, 8, 128, 64, "cpu", permute_pool=True)
    w = w_cpu.to("cuda")
    rng = np.random.default_rng(3)
    n_out = 160
    idx = np.full((w.B, n_out), -1, np.int32)
    cnt = np.zeros((w.B,), np.int32)
    for r in range(w.B):
        c = int(rng.integers(0, n_out + 1)) if r % 7 else 0
        c = min(c, seq[r])
        idx[r, :c] = np.sort(rng.choice(seq[r], size=c, replace=False))
        cnt[r] = c
    p = binding.make_params(w.B, 32, 8, 128, w.max_pages, w.num_phys_pages, 10)
    assert binding.se_decode_num_splits(p) == 1
    ws = binding.alloc_workspace(p, "cuda")
    ti, tc = torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda()
    out, lse = token_decode(w, p, ws, ti, tc)
    assert binding.se_last_device_status(ws) == 0
    check_attend(w_cpu, ti, tc, out, lse)
    assert torch.all(out[0] == 0) and torch.all(torch.isneginf(lse[0]))


def test_token_decode_reports_out_of_range_tokens():
    w_cpu = wl.build("tok", 982, 0, [100, 50], 8, 2, 128, 64, "cpu")
    w = w_cpu.to("cuda")
    idx = torch.tensor([[0, 5, 99, 100, -1, -1, -1, -1] + [-1] * 8, [1, 2, 3, 49] + [-1] * 12], dtype=torch.int32).cuda()
    cnt = torch.tensor([4, 4], dtype=torch.int32).cuda()
    p = binding.make_params(w.B, 8, 2, 128, w.max_pages, w.num_phys_pages, 1)
    ws = binding.alloc_workspace(p, "cuda")
    out, lse = token_decode(w, p, ws, idx, cnt)
    assert binding.se_last_device_status(ws) & binding.SE_DEV_BAD_SELECTION     # token 100 >= length 100
    good = idx.clone()
    good[0, 3] = -1
    cnt2 = torch.tensor([3, 4], dtype=torch.int32).cuda()
    check_attend(w_cpu, good, cnt2, out, lse)                                     # the bad token was skipped


def test_selection_reuse_workload_full_size_sampled():
    w_cpu = wl.omnikv_workload("cuda")           # generated on the GPU, sampled rows go to the host
    w = w_cpu
    st, keys = observe(w)
    rows = [0, 11, 23]
    sub = wl.sub_workload(w, rows)
    s_ref, present, s_gpu = check_scores(sub, keys[rows].clone(), rows=None)
    tok_idx, tok_cnt = select(st, keys, w, 2048, 32)
    check_select(sub, s_ref, present, s_gpu, tok_idx[rows], tok_cnt[rows], 2048, 32)
    w1 = wl.omnikv_workload("cuda", layer=1)
    p = binding.make_params(w.B, w.H_q, w.H_kv, w.D, w.max_pages, w.num_phys_pages, (2048 + 32 + 15) // 16)
    ws = binding.alloc_workspace(p, "cuda")
    out, lse = token_decode(w1, p, ws, tok_idx, tok_cnt)
    assert binding.se_last_device_status(ws) == 0
    check_attend(wl.sub_workload(w1, rows), tok_idx[rows], tok_cnt[rows], out[rows], lse[rows])
