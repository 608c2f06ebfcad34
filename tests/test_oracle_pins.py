"""Pins for the CPU oracle: every check compares it with something that is not itself —
numpy brute force written from the definitions, closed forms, the inequalities and
special cases the paper states, and a library routine (torch SDPA / logsumexp in fp64).
Runs without a GPU."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39068_b200 import workloads as wl
from helpers import (bits_to_f64, dense_attention_np, f32_to_bits, host_arrays,
                     tokens_of_request)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = [int(x) for x in v]
    return out


def random_bits(rng, shape, scale=1.0):
    x = torch.from_numpy(rng.standard_normal(shape).astype(np.float32) * scale)
    return wl.bf16_bits(x.to(torch.bfloat16))


def small_case(seed=0, seq=(37, 16, 1, 50), H_q=4, H_kv=2, D=8, budget=32, **kw):
    w = wl.build("t", 900 + seed, 0, list(seq), H_q, H_kv, D, budget, "cpu", **kw)
    return w, host_arrays(w)


# ---------------------------------------------------------------- O1 page summaries

@pytest.mark.parametrize("permute", [False, True])
def test_meta_matches_bruteforce(permute):
    w, a = small_case(1, permute_pool=permute, poison_tail=True, spare_pages=2)
    sentinel = np.full((w.num_phys_pages, w.H_kv, 2, w.D), 0x7FC0, dtype=np.uint16)
    meta = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=np.zeros(w.B, np.int32),
                             meta=sentinel)
    K = bits_to_f64(a["k"])
    touched = np.zeros(w.num_phys_pages, bool)
    for r in range(w.B):
        L = int(a["seq_lens"][r])
        for b in range((L + 15) // 16):
            pid = a["page_table"][r, b]
            nv = min(16, L - 16 * b)
            touched[pid] = True
            for h in range(w.H_kv):
                np.testing.assert_array_equal(bits_to_f64(meta[pid, h, 0]), K[pid, h, :nv].min(0))
                np.testing.assert_array_equal(bits_to_f64(meta[pid, h, 1]), K[pid, h, :nv].max(0))
    assert np.all(meta[~touched] == 0x7FC0), "pages no request refers to must stay untouched"
    assert (~touched).sum() >= 2


def test_meta_min_below_max_and_idempotent():
    w, a = small_case(2)
    ft = np.zeros(w.B, np.int32)
    m1 = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=ft)
    m2 = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=ft, meta=m1)
    np.testing.assert_array_equal(m1, m2)
    assert np.all(bits_to_f64(m1[:, :, 0]) <= bits_to_f64(m1[:, :, 1]))


def test_meta_incremental_equals_rebuild():
    """Appending one token and updating only its page gives the same summaries as a
    rebuild from scratch (Appendix A, Quest: a new key changes only its own page's summary)."""
    w, a = small_case(3, seq=(33, 48, 16, 5))
    ft = np.zeros(w.B, np.int32)
    grown = a["seq_lens"].copy()
    short = grown - 1
    # request 2 has exactly one full page, so shrinking leaves 15 tokens in that page
    meta_before = oracle.quest_meta(a["k"], a["page_table"], short, first_tok=ft)
    inc = oracle.quest_meta(a["k"], a["page_table"], grown, first_tok=None, meta=meta_before)
    full = oracle.quest_meta(a["k"], a["page_table"], grown, first_tok=ft)
    np.testing.assert_array_equal(inc, full)
    assert not np.array_equal(meta_before, full)


def test_meta_signed_zero_rule():
    k = np.zeros((1, 1, 16, 2), np.uint16)
    k[0, 0, 0, 0] = 0x0000
    k[0, 0, 1, 0] = 0x8000          # -0 after +0
    k[0, 0, 0, 1] = 0x8000
    k[0, 0, 1, 1] = 0x0000          # +0 after -0
    meta = oracle.quest_meta(k, np.array([[0]]), np.array([2]), first_tok=np.array([0]))
    assert meta[0, 0, 0].tolist() == [0x8000, 0x8000]
    assert meta[0, 0, 1].tolist() == [0x0000, 0x0000]


# ---------------------------------------------------------------- O2 page scores

def all_logits(w, a, r, head):
    """z for every stored token of request r and query head `head` (numpy, fp64)."""
    G = w.H_q // w.H_kv
    h = head // G
    qv = bits_to_f64(a["q"][r, head])
    K = bits_to_f64(a["k"])
    toks = tokens_of_request(a["page_table"][r], a["seq_lens"][r], 16)
    z = np.array([K[pid, h, t] @ qv for (_, t, pid) in toks]) / np.sqrt(w.D)
    return toks, z


@pytest.mark.parametrize("cfg", ["small", "config1"])
def test_score_upper_bounds_every_token_logit(cfg):
    """The page score is an upper bound of the logit of every token in the page, for
    every query head (stated below the Quest score equation)."""
    if cfg == "small":
        w, a = small_case(4, seq=(70, 16, 1, 129), H_q=6, H_kv=2, D=16, permute_pool=True)
    else:
        w = wl.config1("cpu")
        a = host_arrays(w)
    meta = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=np.zeros(w.B, np.int32))
    S, P, present = oracle.quest_scores(a["q"], meta, a["page_table"], a["seq_lens"])
    G = w.H_q // w.H_kv
    K = bits_to_f64(a["k"])
    for r in range(w.B):
        L = int(a["seq_lens"][r])
        for head in range(w.H_q):
            toks, z = all_logits(w, a, r, head)
            for (b, t, pid), zz in zip(toks, z):
                assert S[r, head, b] >= zz - 1e-12 * (1 + abs(zz)), (r, head, b, t)
                assert P[r, head // G, b] >= zz - 1e-12 * (1 + abs(zz))
            # and it is not vacuous: it never exceeds sum_c |q_c| * max_t |k_{t,c}| / sqrt(D)
            qabs = np.abs(bits_to_f64(a["q"][r, head]))
            for b in sorted({b for b, _, _ in toks}):
                pid = a["page_table"][r, b]
                nv = min(16, L - 16 * b)
                cap = (qabs * np.abs(K[pid, head // G, :nv]).max(0)).sum() / np.sqrt(w.D)
                assert S[r, head, b] <= cap * (1 + 1e-12)


def test_score_equals_logit_on_single_token_pages():
    """A page with one valid token has m = M = k, so its score is that token's logit."""
    w, a = small_case(5, seq=(17, 33, 1, 49), H_q=4, H_kv=2, D=16, poison_tail=True)
    meta = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=np.zeros(w.B, np.int32))
    S, _, _ = oracle.quest_scores(a["q"], meta, a["page_table"], a["seq_lens"])
    for r in range(w.B):
        L = int(a["seq_lens"][r])
        b = (L - 1) // 16
        for head in range(w.H_q):
            toks, z = all_logits(w, a, r, head)
            assert toks[-1][0] == b and toks[-1][1] == 0
            np.testing.assert_allclose(S[r, head, b], z[-1], rtol=1e-13, atol=1e-13)


def test_score_unit_vector_closed_form():
    """q = s*e_c  ⇒  score = s*M_c/sqrt(D) for s > 0 and s*m_c/sqrt(D) for s < 0."""
    rng = np.random.default_rng(6)
    P_, H_kv, D = 3, 2, 8
    H_q = 4
    meta_f = np.sort(rng.integers(-8, 9, size=(P_, H_kv, 2, D)).astype(np.float32), axis=2)
    meta = f32_to_bits(meta_f)
    page_table = np.array([[2, 0, 1]], np.int32)
    seq = np.array([48], np.int32)
    for c in range(D):
        for s in (2.0, -0.5):
            qf = np.zeros((1, H_q, D), np.float32)
            qf[0, :, c] = s * np.arange(1, H_q + 1)      # a different multiple per head
            S, P, present = oracle.quest_scores(f32_to_bits(qf), meta, page_table, seq)
            for a_ in range(H_q):
                h = a_ // 2
                for b in range(3):
                    pid = page_table[0, b]
                    ext = meta_f[pid, h, 1, c] if s > 0 else meta_f[pid, h, 0, c]
                    np.testing.assert_allclose(S[0, a_, b], s * (a_ + 1) * ext / np.sqrt(D), rtol=1e-14)
            assert present.all()


def test_score_group_reduction_and_scale():
    w, a = small_case(7, H_q=8, H_kv=2, D=16)
    meta = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=np.zeros(w.B, np.int32))
    S, P, present = oracle.quest_scores(a["q"], meta, a["page_table"], a["seq_lens"])
    G = 4
    np.testing.assert_array_equal(P, S.reshape(w.B, 2, G, -1).max(2))
    S2, P2, _ = oracle.quest_scores(a["q"], meta, a["page_table"], a["seq_lens"], sm_scale=0.5)
    np.testing.assert_allclose(S2, S * (0.5 * np.sqrt(16)), rtol=1e-14)
    _, Psum, _ = oracle.quest_scores(a["q"], meta, a["page_table"], a["seq_lens"], group_sum=True)
    np.testing.assert_allclose(Psum, S.reshape(w.B, 2, G, -1).sum(2), rtol=1e-13, atol=1e-13)
    # numpy restatement of the score for one (request, head, page)
    Mf = bits_to_f64(meta)
    qf = bits_to_f64(a["q"])
    for (r, head, b) in [(0, 0, 0), (3, 7, 2), (0, 5, 1)]:
        pid = a["page_table"][r, b]
        h = head // G
        ref = np.maximum(qf[r, head] * Mf[pid, h, 0], qf[r, head] * Mf[pid, h, 1]).sum() / 4.0
        np.testing.assert_allclose(S[r, head, b], ref, rtol=1e-13)
    # pages past the length are not candidates
    for r in range(w.B):
        n_r = (int(a["seq_lens"][r]) + 15) // 16
        assert present[r, :n_r].all() and not present[r, n_r:].any()


def test_quest_example_of_the_paper_shape():
    """Eight tokens in four two-token pages → four summaries → two pages attended."""
    g = read_golden("quest_page_example.txt")
    n, p = g["tokens"][0], g["page_size"][0]
    rng = np.random.default_rng(8)
    D = 4
    k = random_bits(rng, (n // p, 1, p, D))
    v = random_bits(rng, (n // p, 1, p, D))
    q = random_bits(rng, (1, 1, D))
    pt = np.arange(n // p, dtype=np.int32)[None]
    seq = np.array([n], np.int32)
    meta = oracle.quest_meta(k, pt, seq, page_size=p, first_tok=np.array([0]))
    assert meta.shape[0] == g["summaries"][0]
    S, P, present = oracle.quest_scores(q, meta, pt, seq, page_size=p)
    sel, cnt, _ = oracle.topk_pages(P, present, budget=g["selected_pages"][0] * p, page_size=p)
    assert cnt[0, 0] == g["selected_pages"][0]
    Kf, Vf, qf = bits_to_f64(k), bits_to_f64(v), bits_to_f64(q)[0, 0]
    page_scores = [np.maximum(qf * Kf[b, 0].min(0), qf * Kf[b, 0].max(0)).sum() / 2.0 for b in range(4)]
    want = sorted(np.argsort(-np.array(page_scores), kind="stable")[:2].tolist())
    assert sel[0, 0, :2].tolist() == want
    out, lse = oracle.attend(q, k, v, pt, seq, sel, cnt, page_size=p)
    rows = [(b, t) for b in want for t in range(p)]
    o_ref, l_ref = dense_attention_np(qf, np.array([Kf[b, 0, t] for b, t in rows]),
                                      np.array([Vf[b, 0, t] for b, t in rows]), 0.5)
    np.testing.assert_allclose(out[0, 0], o_ref, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], l_ref, rtol=1e-13)


# ---------------------------------------------------------------- O3 top-k

@pytest.mark.parametrize("seed", range(4))
def test_topk_matches_argsort_bruteforce(seed):
    rng = np.random.default_rng(100 + seed)
    B, H, n = 3, 2, 37
    P = rng.standard_normal((B, H, n))
    P[0, 0, 5] = P[0, 0, 9] = P[0, 0, 20] = 10.0        # a tie at the top
    P[1, 1, :] = np.round(P[1, 1, :])                   # many ties everywhere
    present = rng.random((B, n)) > 0.2
    present[2, :] = False
    present[2, [3, 30]] = True                          # fewer candidates than k
    for k in (1, 4, 11, 40):
        sel, cnt, theta = oracle.topk_pages(P, present, budget=16 * k, k_max=k)
        for r in range(B):
            cand = np.nonzero(present[r])[0]
            for h in range(H):
                order = sorted(cand.tolist(), key=lambda b: (-P[r, h, b], b))
                k_eff = min(k, len(cand))
                assert cnt[r, h] == k_eff
                assert sel[r, h, :k_eff].tolist() == sorted(order[:k_eff])
                assert np.all(sel[r, h, k_eff:] == -1)
                if k_eff:
                    assert theta[r, h, 0] == P[r, h, order[k_eff - 1]]
                if k_eff < len(cand):
                    assert theta[r, h, 1] == P[r, h, order[k_eff]]
                else:
                    assert np.isnan(theta[r, h, 1])


def test_topk_budget_rounds_down_to_pages():
    P = np.arange(10, dtype=np.float64)[None, None]
    present = np.ones((1, 10), bool)
    sel, cnt, _ = oracle.topk_pages(P, present, budget=16 * 3 + 15, k_max=8)
    assert cnt[0, 0] == 3 and sel[0, 0, :3].tolist() == [7, 8, 9]


def test_topk_forced_sink_and_recent_pages():
    """The first `sink` and last `recent` pages are always in, outside the budget; the budget is
    spent on the rest (brute force)."""
    rng = np.random.default_rng(200)
    B, H, n = 4, 2, 40
    P = rng.standard_normal((B, H, n))
    seq = np.array([16 * 40, 16 * 23 + 5, 16 * 3, 16 * 9 + 1])
    n_pages = (seq + 15) // 16
    present = np.zeros((B, n), bool)
    for r in range(B):
        present[r, :n_pages[r]] = rng.random(n_pages[r]) > 0.15
    present[0, 0] = False                      # a pruned sink page is simply not there
    for sink, recent, k in [(2, 3, 5), (0, 4, 2), (3, 0, 50), (4, 4, 1)]:
        sel, cnt, theta = oracle.topk_pages(P, present, 16 * k, sink_pages=sink, recent_pages=recent,
                                            seq_lens=seq, k_max=k + sink + recent)
        for r in range(B):
            pres = np.nonzero(present[r])[0]
            forced = [b for b in pres if b < sink or b >= n_pages[r] - recent]
            cand = [b for b in pres if b not in forced]
            for h in range(H):
                best = sorted(cand, key=lambda b: (-P[r, h, b], b))[:k]
                want = sorted(forced + best)
                assert cnt[r, h] == len(want)
                assert sel[r, h, :len(want)].tolist() == want
                assert np.all(sel[r, h, len(want):] == -1)


# ---------------------------------------------------------------- O4 attention

def sdpa_reference(w, a, r):
    """Dense attention of request r over all its stored tokens via torch SDPA in fp64."""
    G = w.H_q // w.H_kv
    toks = tokens_of_request(a["page_table"][r], a["seq_lens"][r], 16)
    K = bits_to_f64(a["k"])
    V = bits_to_f64(a["v"])
    Kd = np.stack([np.stack([K[pid, h, t] for (_, t, pid) in toks]) for h in range(w.H_kv)])
    Vd = np.stack([np.stack([V[pid, h, t] for (_, t, pid) in toks]) for h in range(w.H_kv)])
    qt = torch.from_numpy(bits_to_f64(a["q"][r]))[None, :, None, :]             # [1,H_q,1,D]
    kt = torch.from_numpy(Kd).repeat_interleave(G, 0)[None]
    vt = torch.from_numpy(Vd).repeat_interleave(G, 0)[None]
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt)[0, :, 0].numpy()
    z = (qt @ kt.transpose(-1, -2))[0, :, 0] / np.sqrt(w.D)
    return o, torch.logsumexp(z, -1).numpy()


@pytest.mark.parametrize("kw", [dict(), dict(permute_pool=True, poison_tail=True),
                                dict(prune_fraction=0.3, permute_pool=True)])
def test_budget_covering_everything_equals_dense_attention(kw):
    """With every page selected the result is dense attention (S_i = [i])."""
    w, a = small_case(11, seq=(37, 16, 1, 100), H_q=6, H_kv=2, D=16, budget=16 * 8, **kw)
    res = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget=16 * 8)
    for r in range(w.B):
        o, l = sdpa_reference(w, a, r)
        np.testing.assert_allclose(res["out"][r], o, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(res["lse"][r], l, rtol=1e-12)
        n_present = int((a["page_table"][r, :(int(a["seq_lens"][r]) + 15) // 16] >= 0).sum())
        assert np.all(res["sel_cnt"][r] == n_present)


def test_selected_positions_example_of_the_paper():
    """Reading positions {1,4,8} of an eight-token cache: with one-token pages the page
    list is the position list, and the result is softmax attention over those three."""
    g = read_golden("selected_positions_example.txt")
    n = g["cache_tokens"][0]
    pos = [x - 1 for x in g["read_positions"]]
    rng = np.random.default_rng(12)
    D = 8
    k = random_bits(rng, (n, 1, 1, D))
    v = random_bits(rng, (n, 1, 1, D))
    q = random_bits(rng, (1, 2, D))
    pt = np.arange(n, dtype=np.int32)[None]
    sel = np.array(pos, np.int32)[None, None]
    out, lse = oracle.attend(q, k, v, pt, np.array([n]), sel, np.array([[3]]), page_size=1)
    Kf, Vf, qf = bits_to_f64(k)[:, 0, 0], bits_to_f64(v)[:, 0, 0], bits_to_f64(q)[0]
    for a_ in range(2):
        o_ref, l_ref = dense_attention_np(qf[a_], Kf[pos], Vf[pos], 1 / np.sqrt(D))
        np.testing.assert_allclose(out[0, a_], o_ref, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(lse[0, a_], l_ref, rtol=1e-13)


def test_attention_sparse_subset_matches_numpy_and_gqa_mapping():
    w, a = small_case(13, seq=(90, 40), H_q=8, H_kv=4, D=16, budget=32, permute_pool=True)
    res = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget=32)
    K, V, Q = bits_to_f64(a["k"]), bits_to_f64(a["v"]), bits_to_f64(a["q"])
    for r in range(w.B):
        L = int(a["seq_lens"][r])
        for head in range(w.H_q):
            h = head // 2
            rows = []
            for b in res["sel_idx"][r, h, :res["sel_cnt"][r, h]]:
                pid = a["page_table"][r, b]
                rows += [(pid, t) for t in range(min(16, L - 16 * b))]
            o_ref, l_ref = dense_attention_np(Q[r, head], np.array([K[p_, h, t] for p_, t in rows]),
                                              np.array([V[p_, h, t] for p_, t in rows]), 0.25)
            np.testing.assert_allclose(res["out"][r, head], o_ref, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(res["lse"][r, head], l_ref, rtol=1e-12)


def test_identical_keys_closed_form():
    """All keys equal ⇒ uniform weights: out = mean of V, lse = z + ln(n)."""
    rng = np.random.default_rng(14)
    n_pages, D = 3, 8
    krow = random_bits(rng, (D,))
    k = np.broadcast_to(krow, (n_pages, 1, 16, D)).copy()
    v = random_bits(rng, (n_pages, 1, 16, D))
    q = random_bits(rng, (1, 1, D))
    L = 40
    pt = np.arange(n_pages, dtype=np.int32)[None]
    sel = np.arange(n_pages, dtype=np.int32)[None, None]
    out, lse = oracle.attend(q, k, v, pt, np.array([L]), sel, np.array([[n_pages]]))
    z = bits_to_f64(q)[0, 0] @ bits_to_f64(krow) / np.sqrt(D)
    Vf = bits_to_f64(v).reshape(-1, D)[:L]
    np.testing.assert_allclose(out[0, 0], Vf.mean(0), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse[0, 0], z + np.log(L), rtol=1e-13)


def test_invariant_under_pool_permutation_and_aliasing():
    """Results depend on logical content only: a permuted pool, or private copies of
    aliased prefix pages, change nothing."""
    w, a = small_case(15, seq=(80, 64, 50), H_q=4, H_kv=2, D=16, budget=48, shared_prefix_pages=2)
    res = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget=48)
    assert np.all(a["page_table"][:, :2] == a["page_table"][0, :2])
    # de-alias + permute: give every logical page its own physical page in a shuffled pool
    rng = np.random.default_rng(15)
    slots = [(r, b) for r in range(w.B) for b in range((int(a["seq_lens"][r]) + 15) // 16)]
    perm = rng.permutation(len(slots))
    k2 = np.zeros((len(slots),) + a["k"].shape[1:], np.uint16)
    v2 = np.zeros_like(k2)
    pt2 = np.full_like(a["page_table"], -1)
    for new, (r, b) in zip(perm, slots):
        k2[new] = a["k"][a["page_table"][r, b]]
        v2[new] = a["v"][a["page_table"][r, b]]
        pt2[r, b] = new
    res2 = oracle.decode_step(a["q"], k2, v2, pt2, a["seq_lens"], budget=48)
    np.testing.assert_array_equal(res["sel_idx"], res2["sel_idx"])
    np.testing.assert_array_equal(res["out"], res2["out"])
    np.testing.assert_array_equal(res["lse"], res2["lse"])


def test_empty_and_fully_pruned_requests():
    w, a = small_case(16, seq=(0, 20), H_q=4, H_kv=2, D=8)
    a["page_table"][1, :] = -1
    res = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget=32)
    assert np.all(res["sel_cnt"] == 0)
    assert np.all(res["out"] == 0) and np.all(np.isneginf(res["lse"]))


# ---------------------------------------------------------------- O5 H2O statistic

def test_h2o_mass_sums_to_group_size_and_lands_on_attended_slots():
    w, a = small_case(17, seq=(100, 37), H_q=6, H_kv=2, D=16, budget=48, permute_pool=True,
                      spare_pages=1)
    u0 = np.abs(np.random.default_rng(17).standard_normal((w.num_phys_pages, 2, 16)))
    u = u0.copy()
    res = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget=48, u_accum=u)
    du = u - u0
    assert np.all(du >= 0)
    G = 3
    attended = np.zeros_like(du, bool)
    for r in range(w.B):
        L = int(a["seq_lens"][r])
        for h in range(2):
            mass = 0.0
            for b in res["sel_idx"][r, h, :res["sel_cnt"][r, h]]:
                pid = a["page_table"][r, b]
                nv = min(16, L - 16 * b)
                attended[pid, h, :nv] = True
                mass += du[pid, h, :nv].sum()
            np.testing.assert_allclose(mass, G, rtol=1e-12)
    assert np.all(du[~attended] == 0)
    # the increment is the attention weight itself: recompute one head group by hand
    K, Q = bits_to_f64(a["k"]), bits_to_f64(a["q"])
    r, h = 0, 1
    L = int(a["seq_lens"][r])
    slots = [(a["page_table"][r, b], t) for b in res["sel_idx"][r, h, :res["sel_cnt"][r, h]]
             for t in range(min(16, L - 16 * b))]
    acc = np.zeros(len(slots))
    for head in range(h * G, (h + 1) * G):
        z = np.array([K[p_, h, t] @ Q[r, head] for p_, t in slots]) / 4.0
        acc += np.exp(z - res["lse"][r, head])
    np.testing.assert_allclose([du[p_, h, t] for p_, t in slots], acc, rtol=1e-11)
    # a second step adds on top of the first
    u2 = u.copy()
    oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], budget=48, u_accum=u2)
    np.testing.assert_allclose(u2 - u0, 2 * du, rtol=1e-12, atol=1e-15)
