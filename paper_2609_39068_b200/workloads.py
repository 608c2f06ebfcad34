"""Seeded synthetic inputs for the sparse-decode hot path.

This module only *lays out data*: random bf16 tensors, page tables, context lengths.
It contains none of the method's arithmetic (no min/max summaries, no scores, no
attention) and imports neither the CUDA binding nor the CPU oracle, so both sides
can be fed the very same bits.

Layouts produced (all contiguous):
  q           [B, H_q, D]              bf16
  k_cache     [P_phys, H_kv, 16, D]    bf16   one (page, kv-head) = one contiguous chunk
  v_cache     [P_phys, H_kv, 16, D]    bf16
  page_table  [B, max_pages]           int32  physical page of each logical page, -1 = absent
  seq_lens    [B]                      int32  logical tokens, the current one included
  score_accum [P_phys, H_kv, 16]       fp32   (H2O statistic; only where the workload uses it)

Seeds follow ``1000*config + 16*layer + tensor_id`` with tensor ids
q=0, K=1, V=2, outlier channels=3, lengths=4, permutation=5, prune=6, score_accum=7.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import torch

PAGE = 16

T_Q, T_K, T_V, T_OUTLIER, T_LEN, T_PERM, T_PRUNE, T_ACCUM = range(8)


def _seed(config: int, layer: int, tensor_id: int) -> int:
    return 1000 * config + 16 * layer + tensor_id


def _cpu_gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


@dataclasses.dataclass
class Workload:
    """One decode-step input set for one layer."""
    name: str
    B: int
    H_q: int
    H_kv: int
    D: int
    budget: int                      # token budget of the selection
    max_pages: int                   # row stride of page_table
    num_phys_pages: int
    q: torch.Tensor
    k_cache: torch.Tensor
    v_cache: torch.Tensor
    page_table: torch.Tensor
    seq_lens: torch.Tensor
    score_accum: Optional[torch.Tensor] = None
    page_size: int = PAGE
    notes: str = ""

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv

    @property
    def k_pages(self) -> int:
        return self.budget // self.page_size

    def to(self, device) -> "Workload":
        kw = {}
        for f in dataclasses.fields(self):
            v = getattr(self, f.name)
            kw[f.name] = v.to(device) if isinstance(v, torch.Tensor) else v
        return Workload(**kw)


def _randn_bf16(shape, seed: int, device, scale_channels=None, chunk_rows: int = 4096):
    """N(0,1) rounded to bf16, generated chunk by chunk along dim 0 so that the fp32
    temporary stays small.  ``scale_channels`` = (idx [H_kv, n_out], factor) multiplies
    the listed channels of every token before rounding."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    out = torch.empty(shape, dtype=torch.bfloat16, device=dev)
    n0 = shape[0]
    mult = None
    if scale_channels is not None:
        idx, factor = scale_channels
        H_kv, D = shape[1], shape[-1]
        mult = torch.ones(H_kv, D, dtype=torch.float32)
        for h in range(H_kv):
            mult[h, idx[h]] = factor
        mult = mult.to(dev).view(1, H_kv, 1, D)
    for s in range(0, n0, chunk_rows):
        e = min(n0, s + chunk_rows)
        x = torch.randn((e - s,) + tuple(shape[1:]), generator=g, device=dev, dtype=torch.float32)
        if mult is not None:
            x = x * mult
        out[s:e] = x.to(torch.bfloat16)
    return out


def outlier_channels(config: int, layer: int, H_kv: int, D: int, n_out: int = 4) -> torch.Tensor:
    """``n_out`` distinct channel indices per kv-head, fixed for every token."""
    g = _cpu_gen(_seed(config, layer, T_OUTLIER))
    return torch.stack([torch.randperm(D, generator=g)[:n_out] for _ in range(H_kv)])


def build(
    name: str,
    config: int,
    layer: int,
    seq_lens,
    H_q: int,
    H_kv: int,
    D: int,
    budget: int,
    device="cpu",
    outliers: bool = False,
    permute_pool: bool = False,
    shared_prefix_pages: int = 0,
    prune_fraction: float = 0.0,
    with_score_accum: bool = False,
    max_pages: Optional[int] = None,
    spare_pages: int = 0,
    poison_tail: bool = False,
) -> Workload:
    """Generic builder behind the five named configurations and the small test cases.

    * Pages are dealt to requests in request order; with ``permute_pool`` the physical
      ids are a seeded random permutation of the pool.  Structure (lengths, permutation,
      pruning) never depends on ``layer``; only q/K/V/score_accum values do.
    * ``shared_prefix_pages`` > 0: the first that many logical pages of every request
      map to the same physical pages (a radix-cache style shared prefix).
    * ``prune_fraction`` > 0: a seeded choice keyed on the *physical* page id removes
      that share of pages from the page tables (entry -1); a request's last logical
      page is never removed.
    * ``poison_tail``: token slots past a request's length in its last page are filled
      with large finite values in K and V, so a missing length mask shows up.
    """
    seq = torch.as_tensor(seq_lens, dtype=torch.int64)
    B = int(seq.numel())
    n_pages = (seq + PAGE - 1) // PAGE
    if shared_prefix_pages:
        assert int(n_pages.min()) > shared_prefix_pages, "prefix must be shorter than every request"
    private = n_pages - shared_prefix_pages
    P = int(private.sum()) + shared_prefix_pages + spare_pages
    P = max(P, 1)
    mp = int(max_pages if max_pages is not None else max(int(n_pages.max()), 1))
    assert mp >= int(n_pages.max())

    if permute_pool:
        perm = torch.randperm(P, generator=_cpu_gen(_seed(config, 0, T_PERM)))
    else:
        perm = torch.arange(P)
    page_table = torch.full((B, mp), -1, dtype=torch.int64)
    shared_ids = perm[:shared_prefix_pages]
    cursor = shared_prefix_pages
    for r in range(B):
        n = int(n_pages[r])
        if shared_prefix_pages:
            page_table[r, :shared_prefix_pages] = shared_ids
        cnt = n - shared_prefix_pages
        page_table[r, shared_prefix_pages:n] = perm[cursor:cursor + cnt]
        cursor += cnt

    if prune_fraction > 0.0:
        u = torch.rand(P, generator=_cpu_gen(_seed(config, 0, T_PRUNE)))
        drop_phys = u < prune_fraction
        for r in range(B):
            n = int(n_pages[r])
            if n <= 1:
                continue
            row = page_table[r, : n - 1]
            row[drop_phys[row]] = -1

    chans = None
    if outliers:
        chans = (outlier_channels(config, layer, H_kv, D), 8.0)
    k_cache = _randn_bf16((P, H_kv, PAGE, D), _seed(config, layer, T_K), device, chans)
    v_cache = _randn_bf16((P, H_kv, PAGE, D), _seed(config, layer, T_V), device, chans)
    q = _randn_bf16((B, H_q, 1, D), _seed(config, layer, T_Q), device).view(B, H_q, D)

    if poison_tail:
        for r in range(B):
            L = int(seq[r])
            if L == 0 or L % PAGE == 0:
                continue
            pid = int(page_table[r, (L - 1) // PAGE])
            if pid >= 0:
                k_cache[pid, :, L % PAGE:, :] = 3.0e4
                v_cache[pid, :, L % PAGE:, :] = -3.0e4

    accum = None
    if with_score_accum:
        g = torch.Generator(device=torch.device(device))
        g.manual_seed(_seed(config, layer, T_ACCUM))
        accum = torch.randn((P, H_kv, PAGE), generator=g, device=device, dtype=torch.float32).abs_()

    return Workload(
        name=name, B=B, H_q=H_q, H_kv=H_kv, D=D, budget=budget, max_pages=mp,
        num_phys_pages=P, q=q, k_cache=k_cache, v_cache=v_cache,
        page_table=page_table.to(torch.int32).to(device),
        seq_lens=seq.to(torch.int32).to(device), score_accum=accum,
    )


def _lengths(config: int, layer_independent_seed: int, B: int, lo: int, hi: int) -> torch.Tensor:
    g = _cpu_gen(_seed(config, 0, T_LEN) + layer_independent_seed)
    return torch.randint(lo, hi + 1, (B,), generator=g)


# ---- the five named configurations -------------------------------------------------

def config1(device="cpu", layer: int = 0) -> Workload:
    """Tiny single layer: B=1, 8 q / 2 kv heads, D=64, 2048 tokens, budget 256."""
    return build("config1_tiny", 1, layer, [2048], 8, 2, 64, 256, device)


def config2(device="cpu", layer: int = 0) -> Workload:
    """Llama-3-8B-shaped layer: B=8, 32/8 heads, D=128, 32768 tokens each, budget 2048."""
    return build("config2_llama8b_b8_32k", 2, layer, [32768] * 8, 32, 8, 128, 2048, device,
                 outliers=True)


def config3(device="cpu", layer: int = 0, B: int = 64, lo: int = 4096, hi: int = 65536) -> Workload:
    """Continuous-batching mix: B=64, lengths uniform in [4096, 65536], permuted pool."""
    seq = _lengths(3, 0, B, lo, hi)
    return build("config3_contbatch_b64_mix", 3, layer, seq, 32, 8, 128, 2048, device,
                 outliers=True, permute_pool=True, max_pages=(hi + PAGE - 1) // PAGE)


def config4(device="cpu", layer: int = 0, B: int = 4, length: int = 131072) -> Workload:
    """Long-context eviction decode: B=4, 131072 tokens, budget 4096, H2O statistic on."""
    return build("config4_longctx_h2o", 4, layer, [length] * B, 32, 8, 128, 4096, device,
                 outliers=True, with_score_accum=True)


def config5(device="cpu", layer: int = 0, B: int = 128, lo: int = 8192, hi: int = 32768,
            prefix_tokens: int = 4096) -> Workload:
    """One layer of the 28-layer step: B=128, 28/4 heads (group of 7), lengths uniform in
    [8192, 32768], budget 1024, 4096-token shared prefix aliased, 10 % of pages pruned.
    The page table does not depend on ``layer``; q/K/V do."""
    seq = _lengths(5, 0, B, lo, hi)
    w = build("config5_28layer_b128_gqa7", 5, layer, seq, 28, 4, 128, 1024, device,
              permute_pool=True, shared_prefix_pages=prefix_tokens // PAGE,
              prune_fraction=0.10, max_pages=(hi + PAGE - 1) // PAGE)
    return w


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def h2o_evict_workload(device="cpu", B: int = 64, cached: int = 5120, budget: int = 4096) -> Workload:
    """Periodic decode eviction of an H2O cache: B=64 concurrent requests, each 1024 tokens over its
    4096-token budget (the paper's settings evict every 1024 decode steps), 32/8 heads, D=128,
    pages dealt from a permuted pool, accumulated scores |N(0,1)|."""
    return build("h2o_evict_b64_5120to4096", 6, 0, [cached] * B, 32, 8, 128, budget, device,
                 permute_pool=True, with_score_accum=True)


def omnikv_workload(device="cpu", layer: int = 0, B: int = 24, length: int = 32768) -> Workload:
    """One layer of a selection-reuse step: 24 concurrent requests (the paper's OmniKV concurrency) of
    32768 tokens, 32/8 heads, D=128, 2048 selected + 32 recent tokens.  Layer 0 plays the observation
    layer, layers 1.. the sparse layers that reuse its token set; the page table does not depend on
    ``layer``, q/K/V do."""
    return build("omnikv_reuse_b24_32k", 7, layer, [length] * B, 32, 8, 128, 2048, device, outliers=True,
                 permute_pool=True)


def sub_workload(w: Workload, rows, device="cpu") -> Workload:
    """The requests ``rows`` of ``w`` with their pages gathered into a compact pool of their
    own (physical ids renumbered, aliasing preserved).  Pure data movement: it lets a few
    requests of a multi-gigabyte workload be handed to the CPU without copying the pool."""
    rows = [int(r) for r in rows]
    pt = w.page_table[rows].cpu().to(torch.int64)
    used = torch.unique(pt[pt >= 0])
    remap = torch.full((w.num_phys_pages,), -1, dtype=torch.int64)
    remap[used] = torch.arange(used.numel())
    new_pt = torch.where(pt >= 0, remap[pt.clamp(min=0)], torch.full_like(pt, -1))
    idx = used.to(w.k_cache.device)
    accum = None if w.score_accum is None else w.score_accum[idx].to(device)
    ridx = torch.tensor(rows, device=w.q.device)
    return Workload(
        name=w.name + "_sub%d" % len(rows), B=len(rows), H_q=w.H_q, H_kv=w.H_kv, D=w.D,
        budget=w.budget, max_pages=w.max_pages, num_phys_pages=int(used.numel()),
        q=w.q[ridx].to(device), k_cache=w.k_cache[idx].to(device), v_cache=w.v_cache[idx].to(device),
        page_table=new_pt.to(torch.int32).to(device), seq_lens=w.seq_lens[ridx].to(device),
        score_accum=accum)


def shard_kv_heads(w: Workload, rank: int, world: int) -> Workload:
    """Tensor-parallel shard ``rank`` of ``world``: a contiguous block of kv-heads with their
    query heads.  Page table and lengths are replicated; no step of the path needs data of
    another shard (pure slicing, no arithmetic)."""
    assert w.H_kv % world == 0
    hk = w.H_kv // world
    G = w.H_q // w.H_kv
    ks = slice(rank * hk, (rank + 1) * hk)
    qs = slice(rank * hk * G, (rank + 1) * hk * G)
    return Workload(
        name="%s_tp%dof%d" % (w.name, rank, world), B=w.B, H_q=hk * G, H_kv=hk, D=w.D, budget=w.budget,
        max_pages=w.max_pages, num_phys_pages=w.num_phys_pages, q=w.q[:, qs].contiguous(),
        k_cache=w.k_cache[:, ks].contiguous(), v_cache=w.v_cache[:, ks].contiguous(),
        page_table=w.page_table, seq_lens=w.seq_lens,
        score_accum=None if w.score_accum is None else w.score_accum[:, ks].contiguous())


def bf16_bits(t: torch.Tensor):
    """The raw bf16 bit patterns of ``t`` as a numpy uint16 array on the host."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")
