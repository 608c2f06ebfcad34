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
    st.step(score_accum=u, fused=bool(seed % 2))
    torch.cuda.synchronize()
    assert st.status() == 0, c
    if u is not None:
        compare(w_cpu, st, u_before=w_cpu.score_accum.numpy(), u_after=u.cpu().numpy(), sink_pages=c["sink"],
                recent_pages=c["recent"])
    else:
        compare(w_cpu, st, sink_pages=c["sink"], recent_pages=c["recent"])
