"""Pins for the oracle's H2O retention and eviction: the paper's worked example, numpy brute
force written from the retention equation, the properties the paper states (the window is always
kept, a token that leaves the window competes on its score), and attention over the retained
tokens before and after compaction against an independent numpy softmax.  Runs without a GPU."""
import numpy as np
import pytest

import oracle
from paper_2609_39068_b200 import workloads as wl
from helpers import bits_to_f64, dense_attention_np, host_arrays
from test_oracle_pins import read_golden


def case(seed, seq, H_q=4, H_kv=2, D=8, **kw):
    w = wl.build("h2o", 950 + seed, 0, list(seq), H_q, H_kv, D, 64, "cpu", with_score_accum=True, **kw)
    a = host_arrays(w)
    a["u"] = w.score_accum.numpy().astype(np.float64)
    return w, a


def brute_retain(u_tokens, present, budget, recent):
    """u_tokens [n], present [n] bool -> sorted retained positions, straight from the equation."""
    n = len(u_tokens)
    w = min(recent, budget)
    A = [j for j in range(n) if present[j]]
    W = [j for j in A if j >= n - w]
    rest = [j for j in A if j < n - w]
    rest.sort(key=lambda j: (-u_tokens[j], j))
    return sorted(W + rest[:max(budget - len(W), 0)])


def token_scores(a, r, h, p=16):
    n = int(a["seq_lens"][r])
    u = np.zeros(n)
    present = np.zeros(n, bool)
    for j in range(n):
        pid = int(a["page_table"][r, j // p])
        if pid >= 0:
            present[j] = True
            u[j] = a["u"][pid, h, j % p]
    return u, present


def test_paper_example_budget_four_two_recent():
    g = read_golden("h2o_retention_example.txt")
    budget, recent = g["budget"][0], g["protected_recent"][0]
    # seven cached tokens in one page; scores chosen so that the two best older tokens are 1 and 3
    u = np.zeros((1, 1, 16))
    u[0, 0, :7] = [0.10, 0.90, 0.05, 0.70, 0.20, 0.01, 0.02]
    pt = np.array([[0]], np.int32)
    idx, cnt = oracle.h2o_retain(u, pt, np.array([7], np.int32), budget, recent)
    assert cnt[0, 0] == budget
    assert idx[0, 0].tolist() == [1, 3, 5, 6]          # two heavy hitters + the two most recent tokens
    assert len([j for j in idx[0, 0] if j < 5]) == g["older_slots"][0]


@pytest.mark.parametrize("budget,recent", [(32, 8), (32, 0), (32, 32), (32, 100), (16, 5), (200, 10), (1, 1)])
@pytest.mark.parametrize("prune", [0.0, 0.3])
def test_retain_matches_bruteforce(budget, recent, prune):
    w, a = case(1, (70, 33, 16, 1, 120), permute_pool=True, prune_fraction=prune)
    idx, cnt = oracle.h2o_retain(a["u"], a["page_table"], a["seq_lens"], budget, recent)
    for r in range(w.B):
        for h in range(w.H_kv):
            u, present = token_scores(a, r, h)
            want = brute_retain(u, present, budget, recent)
            got = idx[r, h, :cnt[r, h]].tolist()
            assert got == want
            assert np.all(idx[r, h, cnt[r, h]:] == -1)
            assert cnt[r, h] == min(budget, int(present.sum()))


def test_ties_go_to_the_lower_position_and_window_is_kept():
    u = np.full((2, 1, 16), 0.5)
    pt = np.array([[0, 1]], np.int32)
    idx, cnt = oracle.h2o_retain(u, pt, np.array([20], np.int32), 6, 2)
    assert idx[0, 0, :cnt[0, 0]].tolist() == [0, 1, 2, 3, 18, 19]
    # the window is kept even when its scores are the lowest
    u[1, 0, 2:4] = -1.0
    idx, cnt = oracle.h2o_retain(u, pt, np.array([20], np.int32), 6, 2)
    assert idx[0, 0, :cnt[0, 0]].tolist() == [0, 1, 2, 3, 18, 19]


def test_token_leaving_the_window_competes_on_its_score():
    # step i: 6 tokens, budget 4, window 2 -> token 4 is protected although its score is lowest
    u = np.zeros((1, 1, 16))
    u[0, 0, :6] = [0.9, 0.1, 0.8, 0.2, 0.0, 0.3]
    pt = np.array([[0]], np.int32)
    idx, _ = oracle.h2o_retain(u, pt, np.array([6], np.int32), 4, 2)
    assert idx[0, 0].tolist() == [0, 2, 4, 5]
    # compact, append one token: the old token 4 (now position 2) has left the window and is
    # evicted on its score, while the heavy hitters stay
    k = np.zeros((1, 1, 16, 8), np.uint16)
    _, _, u2, new_len = oracle.h2o_compact(k, k, u, pt, idx, np.array([[4]], np.int32))
    assert new_len.tolist() == [4] and u2[0, 0, :4].tolist() == [0.9, 0.8, 0.0, 0.3]
    u2[0, 0, 4] = 0.05                      # the new token (its score after its first step)
    idx2, _ = oracle.h2o_retain(u2, pt, np.array([5], np.int32), 4, 2)
    assert idx2[0, 0].tolist() == [0, 1, 3, 4]


def test_compaction_is_a_gather_and_preserves_attention():
    w, a = case(2, (90, 40, 17), permute_pool=True)
    budget, recent = 32, 8
    idx, cnt = oracle.h2o_retain(a["u"], a["page_table"], a["seq_lens"], budget, recent)
    k2, v2, u2, new_lens = oracle.h2o_compact(a["k"], a["v"], a["u"], a["page_table"], idx, cnt)
    K, V, K2, V2 = (bits_to_f64(x) for x in (a["k"], a["v"], k2, v2))
    q = bits_to_f64(a["q"])
    scale = 1.0 / np.sqrt(w.D)
    G = w.H_q // w.H_kv
    assert new_lens.tolist() == [min(budget, int(n)) for n in a["seq_lens"]]
    for r in range(w.B):
        for h in range(w.H_kv):
            rows = idx[r, h, :cnt[r, h]]
            src = [(int(a["page_table"][r, j // 16]), j % 16) for j in rows]
            dst = [(int(a["page_table"][r, i // 16]), i % 16) for i in range(len(rows))]
            for (ps, ts), (pd, td) in zip(src, dst):
                assert np.array_equal(k2[pd, h, td], a["k"][ps, h, ts])
                assert np.array_equal(v2[pd, h, td], a["v"][ps, h, ts])
                assert u2[pd, h, td] == a["u"][ps, h, ts]
            # attention over the retained tokens of the old cache == dense attention over the new one
            Ks = np.stack([K[ps, h, ts] for ps, ts in src]); Vs = np.stack([V[ps, h, ts] for ps, ts in src])
            Kd = np.stack([K2[pd, h, td] for pd, td in dst]); Vd = np.stack([V2[pd, h, td] for pd, td in dst])
            for g in range(G):
                o1, l1 = dense_attention_np(q[r, h * G + g], Ks, Vs, scale)
                o2, l2 = dense_attention_np(q[r, h * G + g], Kd, Vd, scale)
                assert np.array_equal(o1, o2) and l1 == l2
    # the oracle's own attention on the compacted cache, all pages selected, agrees as well
    n_pages = (new_lens + 15) // 16
    sel = np.full((w.B, w.H_kv, w.max_pages), -1, np.int32)
    scnt = np.zeros((w.B, w.H_kv), np.int32)
    for r in range(w.B):
        sel[r, :, :n_pages[r]] = np.arange(n_pages[r])
        scnt[r, :] = n_pages[r]
    out, lse = oracle.attend(a["q"], k2, v2, a["page_table"], new_lens, sel, scnt)
    for r in range(w.B):
        for h in range(w.H_kv):
            rows = idx[r, h, :cnt[r, h]]
            Ks = np.stack([K[int(a["page_table"][r, j // 16]), h, j % 16] for j in rows])
            Vs = np.stack([V[int(a["page_table"][r, j // 16]), h, j % 16] for j in rows])
            for g in range(G):
                o, l = dense_attention_np(q[r, h * G + g], Ks, Vs, scale)
                assert np.allclose(out[r, h * G + g], o, rtol=1e-12, atol=1e-12)
                assert abs(lse[r, h * G + g] - l) < 1e-12


def test_nothing_to_evict_is_the_identity():
    w, a = case(3, (20, 5))
    idx, cnt = oracle.h2o_retain(a["u"], a["page_table"], a["seq_lens"], 64, 4)
    assert [cnt[r, 0] for r in range(2)] == [20, 5]
    assert idx[0, 0, :20].tolist() == list(range(20))
    k2, v2, u2, new_lens = oracle.h2o_compact(a["k"], a["v"], a["u"], a["page_table"], idx, cnt)
    assert np.array_equal(k2, a["k"]) and np.array_equal(v2, a["v"]) and np.array_equal(u2, a["u"])
    assert new_lens.tolist() == [20, 5]
