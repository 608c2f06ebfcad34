"""Independent numpy re-derivations used to pin the oracle, and the comparison rules
used to check the CUDA path against it.  Nothing here calls the oracle's C routines or
the CUDA library."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_39068_b200 import workloads as wl


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) → float64, exactly."""
    w = bits.astype(np.uint32) << np.uint32(16)
    return w.view(np.float32).astype(np.float64)


def f32_to_bits(x: np.ndarray) -> np.ndarray:
    """float values that are exactly representable in bf16 → their bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = x.view(np.uint32)
    assert np.all((w & np.uint32(0xFFFF)) == 0), "value not representable in bf16"
    return (w >> np.uint32(16)).astype(np.uint16)


def host_arrays(w: wl.Workload):
    """numpy views of a workload: bf16 tensors as uint16 bit patterns."""
    return dict(
        q=wl.bf16_bits(w.q), k=wl.bf16_bits(w.k_cache), v=wl.bf16_bits(w.v_cache),
        page_table=w.page_table.cpu().numpy().astype(np.int32),
        seq_lens=w.seq_lens.cpu().numpy().astype(np.int32),
    )


def tokens_of_request(page_table_row, length, p):
    """[(logical page, token-in-page, physical page)] of every stored token of a request."""
    out = []
    for j in range(int(length)):
        b, t = j // p, j % p
        pid = int(page_table_row[b])
        if pid >= 0:
            out.append((b, t, pid))
    return out


def dense_attention_np(qv, K, V, scale):
    """Textbook softmax attention of one query vector over rows of K, V (float64)."""
    z = (K @ qv) * scale
    m = z.max()
    e = np.exp(z - m)
    return (e[:, None] * V).sum(0) / e.sum(), m + np.log(e.sum())


def check_selection(sel_gpu, cnt_gpu, P_oracle, present, budget, p=16, rel_band=1e-5,
                    sink_pages=0, recent_pages=0, seq_lens=None):
    """Selected-page rule.  Forced pages (first ``sink_pages`` / last ``recent_pages`` logical pages
    of a request, when present) must all be in the set.  Among the other present pages, with theta
    the oracle's k_eff-th largest score and eps = rel_band*|theta|, the set must hold exactly k_eff
    of them, every page scoring above theta+eps and none scoring below theta-eps.
    Returns the number of (request, head) rows whose set differs from the strict top-k."""
    B, H, n = P_oracle.shape
    k = budget // p
    differing = 0
    for r in range(B):
        pres = np.nonzero(present[r])[0]
        n_r = n if seq_lens is None else (int(seq_lens[r]) + p - 1) // p
        is_forced = (pres < sink_pages) | ((pres >= n_r - recent_pages) & (pres < n_r))
        forced = set(pres[is_forced].tolist())
        cand = pres[~is_forced]
        for h in range(H):
            k_eff = min(k, len(cand))
            total = k_eff + len(forced)
            assert int(cnt_gpu[r, h]) == total, (r, h, int(cnt_gpu[r, h]), total)
            row = np.asarray(sel_gpu[r, h])
            got = row[:total]
            assert np.all(row[total:] == -1), "padding must be -1"
            if total == 0:
                continue
            assert len(set(got.tolist())) == total, "duplicate pages selected"
            assert np.all(present[r][got]), "absent page selected"
            gs = set(got.tolist())
            assert forced <= gs, (r, h, "forced pages missing", sorted(forced - gs)[:5])
            gs -= forced
            if k_eff == 0:
                assert not gs
                continue
            s = P_oracle[r, h]
            order = cand[np.lexsort((cand, -s[cand]))]
            strict = set(order[:k_eff].tolist())
            theta = s[order[k_eff - 1]]
            eps = rel_band * abs(theta)
            must = set(cand[s[cand] > theta + eps].tolist())
            never = set(cand[s[cand] < theta - eps].tolist())
            assert must <= gs, (r, h, "missing pages above the band", sorted(must - gs)[:5])
            assert not (gs & never), (r, h, "pages below the band", sorted(gs & never)[:5])
            if gs != strict:
                differing += 1
    return differing


def to_torch_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
