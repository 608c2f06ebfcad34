"""Pins for the oracle's OmniKV-style path (observation-layer token scores, token top-k, reuse
attention): numpy brute force from the equations, the paper's {1,4,8} example, dense equivalence
against torch SDPA, and agreement with the page-granular attention (pinned elsewhere) when the
token set is exactly the tokens of the selected pages.  Runs without a GPU."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39068_b200 import workloads as wl
from helpers import bits_to_f64, dense_attention_np, host_arrays
from test_oracle_pins import read_golden


def case(seed, seq, H_q=4, H_kv=2, D=8, **kw):
    w = wl.build("tok", 970 + seed, 0, list(seq), H_q, H_kv, D, 64, "cpu", **kw)
    return w, host_arrays(w)


def test_token_scores_match_bruteforce():
    w, a = case(1, (37, 16, 1, 50), permute_pool=True, prune_fraction=0.3)
    s, present = oracle.token_scores(a["q"], a["k"], a["page_table"], a["seq_lens"])
    q, K = bits_to_f64(a["q"]), bits_to_f64(a["k"])
    G = w.H_q // w.H_kv
    scale = 1.0 / np.sqrt(w.D)
    for r in range(w.B):
        n = int(a["seq_lens"][r])
        for j in range(s.shape[1]):
            pid = int(a["page_table"][r, j // 16]) if j < n else -1
            assert present[r, j] == (pid >= 0)
            if pid >= 0:
                z = [scale * float(q[r, h * G + g] @ K[pid, h, j % 16]) for h in range(w.H_kv) for g in range(G)]
                assert abs(s[r, j] - max(z)) < 1e-12
            else:
                assert s[r, j] == 0.0


@pytest.mark.parametrize("budget,recent", [(8, 0), (8, 3), (5, 40), (100, 2), (1, 1)])
def test_token_topk_matches_argsort(budget, recent):
    rng = np.random.default_rng(5)
    B, n = 4, 64
    s = np.round(rng.standard_normal((B, n)) * 4) / 4          # ties on purpose
    present = rng.random((B, n)) > 0.2
    lens = np.array([64, 33, 1, 50], np.int32)
    idx, cnt, theta = oracle.token_topk(s, present, lens, budget, recent)
    for r in range(B):
        L = int(lens[r])
        W = [j for j in range(L) if present[r, j] and j >= L - recent]
        cand = [j for j in range(L) if present[r, j] and j < L - recent]
        cand.sort(key=lambda j: (-s[r, j], j))
        want = sorted(W + cand[:budget])
        assert idx[r, :cnt[r]].tolist() == want and np.all(idx[r, cnt[r]:] == -1)
        if cand and budget:
            assert theta[r] == s[r, cand[min(budget, len(cand)) - 1]]


def test_paper_example_positions_1_4_8_reused_by_two_layers():
    g = read_golden("omnikv_reuse_example.txt")
    pos0 = [x - 1 for x in g["observed_positions"]]             # 0-based
    # an eight-token cache; the observation layer's scores are made to peak at the three positions
    w, a = case(2, (8,), H_q=2, H_kv=1, D=8)
    s = np.zeros((1, 16))
    s[0, pos0] = [3.0, 2.0, 1.0]
    present = np.zeros((1, 16), bool)
    present[0, :8] = True
    idx, cnt, _ = oracle.token_topk(s, present, a["seq_lens"], 3)
    assert idx[0, :cnt[0]].tolist() == pos0
    # every associated sparse layer reads those positions from its own cache
    for layer in range(g["sparse_layers"][0]):
        wl_l = wl.build("tok", 972, layer + 1, [8], 2, 1, 8, 64, "cpu")
        al = host_arrays(wl_l)
        out, lse = oracle.token_attend(al["q"], al["k"], al["v"], al["page_table"], al["seq_lens"], idx, cnt)
        q, K, V = bits_to_f64(al["q"]), bits_to_f64(al["k"]), bits_to_f64(al["v"])
        pid = int(al["page_table"][0, 0])
        for h in range(2):
            o, l = dense_attention_np(q[0, h], K[pid, 0, pos0], V[pid, 0, pos0], 1.0 / np.sqrt(8))
            assert np.allclose(out[0, h], o, rtol=1e-13, atol=1e-13) and abs(lse[0, h] - l) < 1e-13


def test_token_attend_all_tokens_equals_sdpa():
    w, a = case(3, (45, 20), H_q=4, H_kv=2, D=16, permute_pool=True)
    n_out = 48
    idx = np.full((w.B, n_out), -1, np.int32)
    cnt = np.array(a["seq_lens"], np.int32)
    for r in range(w.B):
        idx[r, :cnt[r]] = np.arange(cnt[r])
    out, lse = oracle.token_attend(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], idx, cnt)
    q, K, V = (torch.from_numpy(bits_to_f64(x)) for x in (a["q"], a["k"], a["v"]))
    G = w.H_q // w.H_kv
    for r in range(w.B):
        n = int(cnt[r])
        pids = torch.from_numpy(a["page_table"][r, :(n + 15) // 16].astype(np.int64))
        for h in range(w.H_kv):
            Kr = K[pids, h].reshape(-1, w.D)[:n]
            Vr = V[pids, h].reshape(-1, w.D)[:n]
            qq = q[r, h * G:(h + 1) * G]
            ref = torch.nn.functional.scaled_dot_product_attention(qq[None], Kr[None], Vr[None])[0]
            assert np.allclose(out[r, h * G:(h + 1) * G], ref.numpy(), rtol=1e-12, atol=1e-12)
            ref_lse = torch.logsumexp(qq @ Kr.T / np.sqrt(w.D), dim=1)
            assert np.allclose(lse[r, h * G:(h + 1) * G], ref_lse.numpy(), rtol=1e-12, atol=1e-12)


def test_token_attend_agrees_with_page_attend_on_whole_pages():
    w, a = case(4, (70, 33), H_q=4, H_kv=2, D=8, permute_pool=True)
    pages = [[0, 2, 4], [1, 2]]                               # same pages for every head of a request
    sel = np.full((w.B, w.H_kv, 4), -1, np.int32)
    scnt = np.zeros((w.B, w.H_kv), np.int32)
    idx = np.full((w.B, 64), -1, np.int32)
    cnt = np.zeros((w.B,), np.int32)
    for r, pg in enumerate(pages):
        sel[r, :, :len(pg)] = pg
        scnt[r, :] = len(pg)
        toks = [j for b in pg for j in range(16 * b, min(16 * b + 16, int(a["seq_lens"][r])))]
        idx[r, :len(toks)] = toks
        cnt[r] = len(toks)
    o1, l1 = oracle.attend(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], sel, scnt)
    o2, l2 = oracle.token_attend(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], idx, cnt)
    assert np.allclose(o1, o2, rtol=1e-13, atol=1e-13) and np.allclose(l1, l2, rtol=1e-13, atol=1e-13)


def test_token_attend_skips_absent_tokens_and_empty_sets():
    w, a = case(5, (40, 10), prune_fraction=0.5, permute_pool=True)
    idx = np.full((2, 8), -1, np.int32)
    idx[0, :5] = [0, 17, 20, 39, 45]                          # 45 lies past the length
    cnt = np.array([5, 0], np.int32)
    out, lse = oracle.token_attend(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], idx, cnt)
    assert np.all(out[1] == 0) and np.all(np.isneginf(lse[1]))
    q, K, V = bits_to_f64(a["q"]), bits_to_f64(a["k"]), bits_to_f64(a["v"])
    live = [j for j in (0, 17, 20, 39) if a["page_table"][0, j // 16] >= 0]
    for h_q in range(w.H_q):
        h = h_q // (w.H_q // w.H_kv)
        if not live:
            assert np.isneginf(lse[0, h_q])
            continue
        Ks = np.stack([K[a["page_table"][0, j // 16], h, j % 16] for j in live])
        Vs = np.stack([V[a["page_table"][0, j // 16], h, j % 16] for j in live])
        o, l = dense_attention_np(q[0, h_q], Ks, Vs, 1.0 / np.sqrt(w.D))
        assert np.allclose(out[0, h_q], o, rtol=1e-13, atol=1e-13) and abs(lse[0, h_q] - l) < 1e-13
