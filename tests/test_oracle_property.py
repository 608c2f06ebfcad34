"""Randomised pins for the oracle's three selection rules (page top-k, H2O retained set, token top-k):
hypothesis draws small cases with many ties, absent entries and odd sizes, and each result is
compared with a brute-force restatement of the rule.  Runs without a GPU."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle


def _scores(draw, n, levels):
    return np.array(draw(st.lists(st.integers(-levels, levels), min_size=n, max_size=n)), dtype=np.float64) / 4.0


@st.composite
def page_case(draw):
    n = draw(st.integers(1, 40))
    s = _scores(draw, n, draw(st.integers(0, 6)))
    present = np.array(draw(st.lists(st.booleans(), min_size=n, max_size=n)), dtype=bool)
    n_r = draw(st.integers(0, n))
    present[n_r:] = False
    return s, present, n_r, draw(st.integers(1, 12)), draw(st.integers(0, 3)), draw(st.integers(0, 3))


@settings(max_examples=150, deadline=None)
@given(page_case())
def test_page_topk_rule(case):
    s, present, n_r, k, sink, recent = case
    n = len(s)
    k_max = k + sink + recent
    idx, cnt, _ = oracle.topk_pages(s[None, None, :], present[None, :], 16 * k, k_max=k_max, sink_pages=sink,
                                    recent_pages=recent, seq_lens=np.array([16 * n_r], np.int32))
    forced = [b for b in range(n_r) if present[b] and (b < sink or b >= n_r - recent)]
    cand = [b for b in range(n) if present[b] and b not in forced]
    cand.sort(key=lambda b: (-s[b], b))
    want = sorted(forced + cand[:k])
    assert idx[0, 0, :cnt[0, 0]].tolist() == want
    assert np.all(idx[0, 0, cnt[0, 0]:] == -1)


@st.composite
def token_case(draw):
    pages = draw(st.integers(1, 5))
    n = draw(st.integers(1, 16 * pages))
    u = _scores(draw, 16 * pages, draw(st.integers(0, 5)))
    absent = np.array(draw(st.lists(st.booleans(), min_size=pages, max_size=pages)), dtype=bool)
    return pages, n, u, absent, draw(st.integers(1, 24)), draw(st.integers(0, 24))


@settings(max_examples=150, deadline=None)
@given(token_case())
def test_h2o_retention_rule(case):
    pages, n, u, absent, budget, recent = case
    pt = np.where(absent, -1, np.arange(pages)).astype(np.int32)[None, :]
    idx, cnt = oracle.h2o_retain(u.reshape(pages, 1, 16), pt, np.array([n], np.int32), budget, recent)
    w = min(recent, budget)
    A = [j for j in range(n) if not absent[j // 16]]
    W = [j for j in A if j >= n - w]
    rest = sorted((j for j in A if j < n - w), key=lambda j: (-u[j], j))
    want = sorted(W + rest[:budget - len(W)])
    assert idx[0, 0, :cnt[0, 0]].tolist() == want and cnt[0, 0] == min(budget, len(A))


@settings(max_examples=150, deadline=None)
@given(token_case())
def test_token_topk_rule(case):
    pages, n, s, absent, budget, recent = case
    present = np.repeat(~absent, 16)[None, :]
    idx, cnt, theta = oracle.token_topk(s[None, :], present, np.array([n], np.int32), budget, recent)
    A = [j for j in range(n) if present[0, j]]
    W = [j for j in A if j >= n - recent]
    rest = sorted((j for j in A if j < n - recent), key=lambda j: (-s[j], j))
    want = sorted(W + rest[:budget])
    assert idx[0, :cnt[0]].tolist() == want
    if rest:
        assert theta[0] == s[rest[min(budget, len(rest)) - 1]]
