"""Seeded random shapes through the whole decode step (summaries, selection, attention, optionally the
H2O statistic and forced pages) against the CPU oracle: a sweep over combinations no hand-written
case lists.  Every case is reproducible from its seed."""
import numpy as np
import pytest
import torch

from paper_2609_39068_b200 import binding, workloads as wl
from test_gpu_parity import compare

pytestmark = pytest.mark.gpu


def draw_case(seed):
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.choice([1, 2, 3, 4, 8]))
    G = int(rng.integers(1, 9))
    B = int(rng.integers(1, 7))
    shape = rng.choice(["short", "mixed", "long"])
    hi = {"short": 80, "mixed": 1500, "long": 6000}[shape]
    seq = [int(x) for x in rng.integers(1, hi + 1, size=B)]
    if rng.random() < 0.2:
        seq[int(rng.integers(0, B))] = 0                      # a padding slot
    budget = 16 * int(rng.integers(1, 1 + max(1, min(200, max(seq) // 16 + 3))))
    kw = dict(permute_pool=bool(rng.random() < 0.7), poison_tail=True,
              prune_fraction=float(rng.choice([0.0, 0.0, 0.15, 0.5])),
              outliers=bool(rng.random() < 0.3), with_score_accum=bool(rng.random() < 0.4),
              spare_pages=int(rng.integers(0, 4)))
    if min(seq) > 16 * 12 and rng.random() < 0.3 and kw["prune_fraction"] == 0.0:
        kw["shared_prefix_pages"] = int(rng.integers(1, 10))
        kw["with_score_accum"] = False                         # no aliasing under the H2O epilogue
    sink, recent = (int(rng.integers(0, 3)), int(rng.integers(0, 4))) if rng.random() < 0.3 else (0, 0)
    return dict(seq=seq, H_q=H_kv * G, H_kv=H_kv, D=D, budget=budget, kw=kw, sink=sink, recent=recent)


@pytest.mark.parametrize("seed", range(40))
def test_random_shapes(seed):
    c = draw_case(seed)
    w_cpu = wl.build("fuzz%d" % seed, 700 + seed % 50, 0, c["seq"], c["H_q"], c["H_kv"], c["D"], c["budget"],
                     "cpu", **c["kw"])
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w, sink_pages=c["sink"], recent_pages=c["recent"])
    st.rebuild_meta()
    u = w.score_accum.clone() if w.score_accum is not None else None
    st.step(score_accum=u, fused=bool(seed % 2))       # se_decode_step, or the three separate calls
    torch.cuda.synchronize()
    assert st.status() == 0, c
    if u is not None:
        compare(w_cpu, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy(), sink_pages=c["sink"],
                recent_pages=c["recent"])
    else:
        compare(w_cpu, st, sink_pages=c["sink"], recent_pages=c["recent"])


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_many_requests(seed):
    """The same sweep with up to 200 requests, so that every launch plan (cluster per pair, warp splits and
    the merge kernel, two warps per pair, one warp per pair) meets random shapes, not only the listed ones."""
    rng = np.random.default_rng(50000 + seed)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.choice([1, 2, 3, 4, 8]))
    G = int(rng.integers(1, 9))
    B = min(int(rng.choice([9, 20, 37, 50, 74, 75, 99, 120, 150, 200])), 1300 // H_kv)
    hi = {"short": 80, "mixed": 900, "long": 3000}[str(rng.choice(["short", "mixed", "long"]))]
    seq = [int(x) for x in rng.integers(1, hi + 1, size=B)]
    if rng.random() < 0.3:
        seq[int(rng.integers(0, B))] = 0
    budget = 16 * int(rng.integers(1, 1 + max(1, min(120, max(seq) // 16 + 3))))
    kw = dict(permute_pool=bool(rng.random() < 0.7), poison_tail=True,
              prune_fraction=float(rng.choice([0.0, 0.0, 0.15, 0.5])),
              outliers=bool(rng.random() < 0.3), with_score_accum=bool(rng.random() < 0.4),
              spare_pages=int(rng.integers(0, 4)))
    sink, recent = (int(rng.integers(0, 3)), int(rng.integers(0, 4))) if rng.random() < 0.3 else (0, 0)
    w_cpu = wl.build("fuzzmany%d" % seed, 600 + seed, 0, seq, H_kv * G, H_kv, D, budget, "cpu", **kw)
    w = w_cpu.to("cuda")
    st = binding.DecodeState(w, sink_pages=sink, recent_pages=recent)
    st.rebuild_meta()
    u = w.score_accum.clone() if w.score_accum is not None else None
    st.step(score_accum=u, fused=bool(seed % 2))
    torch.cuda.synchronize()
    assert st.status() == 0
    if u is not None:
        compare(w_cpu, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy(), sink_pages=sink,
                recent_pages=recent)
    else:
        compare(w_cpu, st, sink_pages=sink, recent_pages=recent)


@pytest.mark.parametrize("seed", range(20))
def test_random_h2o_evictions(seed):
    from test_gpu_h2o import check_retain
    import oracle
    from helpers import host_arrays
    rng = np.random.default_rng(2000 + seed)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.choice([1, 2, 4]))
    B = int(rng.integers(1, 5))
    seq = [int(x) for x in rng.integers(1, 3000, size=B)]
    budget = int(rng.integers(1, 1500))
    recent = int(rng.integers(0, 1.2 * budget + 2))
    w_cpu = wl.build("fz", 750 + seed, 0, seq, H_kv * int(rng.integers(1, 5)), H_kv, D, 64, "cpu",
                     permute_pool=True, with_score_accum=True)
    levels = int(rng.choice([0, 2, 16]))
    if levels:
        w_cpu.score_accum = torch.round(w_cpu.score_accum * levels) / levels
    w, p, ws, keep_idx, keep_cnt = check_retain(w_cpu, budget, recent)
    a = host_arrays(w_cpu)
    k_ref, v_ref, u_ref, len_ref = oracle.h2o_compact(a["k"], a["v"], w_cpu.score_accum.numpy().astype(np.float64),
                                                      a["page_table"], keep_idx.cpu().numpy(), keep_cnt.cpu().numpy())
    new_lens = torch.zeros((w.B,), dtype=torch.int32, device="cuda")
    binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt, new_lens, ws)
    torch.cuda.synchronize()
    assert binding.se_last_device_status(ws) == 0
    assert np.array_equal(new_lens.cpu().numpy(), len_ref)
    assert np.array_equal(wl.bf16_bits(w.k_cache), k_ref) and np.array_equal(wl.bf16_bits(w.v_cache), v_ref)
    assert np.array_equal(w.score_accum.cpu().numpy().astype(np.float64), u_ref)


@pytest.mark.parametrize("seed", range(20))
def test_random_selection_reuse(seed):
    from test_gpu_token import observe, check_scores, select, check_select, token_decode, check_attend
    rng = np.random.default_rng(3000 + seed)
    D = int(rng.choice([64, 128]))
    H_kv = int(rng.choice([1, 2, 4]))
    G = int(rng.integers(1, 9))
    B = int(rng.integers(1, 5))
    seq = [int(x) for x in rng.integers(1, 2500, size=B)]
    prune = float(rng.choice([0.0, 0.2]))
    budget, recent = int(rng.integers(0, 600)), int(rng.integers(0, 40))
    if budget + recent == 0:
        budget = 1
    w_cpu = wl.build("fz", 760 + seed, 0, seq, H_kv * G, H_kv, D, 64, "cpu", permute_pool=True, prune_fraction=prune,
                     poison_tail=True)
    w = w_cpu.to("cuda")
    st, keys = observe(w)
    s_ref, present, s_gpu = check_scores(w_cpu, keys)
    tok_idx, tok_cnt = select(st, keys, w, budget, recent)
    check_select(w_cpu, s_ref, present, s_gpu, tok_idx, tok_cnt, budget, recent)
    w1_cpu = wl.build("fz", 760 + seed, 1, seq, H_kv * G, H_kv, D, 64, "cpu", permute_pool=True, prune_fraction=prune,
                      poison_tail=True)
    w1 = w1_cpu.to("cuda")
    p = binding.make_params(w.B, H_kv * G, H_kv, D, w.max_pages, w.num_phys_pages, (budget + recent + 15) // 16)
    ws = binding.alloc_workspace(p, "cuda")
    out, lse = token_decode(w1, p, ws, tok_idx, tok_cnt)
    assert binding.se_last_device_status(ws) == 0
    check_attend(w1_cpu, tok_idx, tok_cnt, out, lse)
