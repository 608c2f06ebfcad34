#!/usr/bin/env python
"""Benchmark of the sparse decode-attention hot path.

A *step* is one pass of the whole path over one batch of synthetic requests, per layer: summary of
the page holding each request's newest token -> page scores -> top-k -> attention over the selected
pages, LSE merge, optional H2O statistic.  One call does it all: ``se_decode_step`` (the library
picks the launch plan from the shape).  The default workload is the continuous-batching mix
(config 3: 64 requests, 4096..65536 tokens, 32/8 heads, D=128, budget 2048, page tables permuted over
one pool); ``--config`` picks another one, and the default run also times the other four configs
briefly (``other_configs`` in the JSON line).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

N > 1: one rank per GPU (started by the driver with torch.distributed.run, or by this script itself
when it is called without a rank environment); every rank runs the same shape on its own data - the
path shards by request / kv-head without any collective - so scaling is weak.  Rank 0 prints ONE JSON
line.

Timing follows the paper's protocol (Experimental Settings, "Measurement Protocol"): one discarded
run, then three windows, each 32 untimed replays followed by K/3 timed ones, CUDA events on the
launching stream, host synchronisation only at window boundaries.  Cold L2 either by construction
(inputs larger than L2, or R independent instances replayed round-robin so that R steps touch at
least four times the L2) or, for the tiny config, by a flush between steps.
"""
from __future__ import annotations

import argparse
import ctypes
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2609_39068_b200 import workloads as wl

METRIC = "sparse_decode_us_per_step"
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
WINDOW_WARMUP = 32                     # untimed replays in front of every timed window

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised in profiles/
# (profiles/full_capture_config3_b40.md: a 40-request capture scaled to the full launch by the pages processed;
# null where no capture of that workload exists)
NCU_TRAFFIC_BYTES = {"config3_contbatch_b64_mix": 543.8e6}          # decode_duo_kernel: 339.89 MB x 65536 / 40960
NCU_TRAFFIC_BYTES_SCORE = {"config3_contbatch_b64_mix": 577.6e6}    # score_kernel: 200.28 MB x 137094 / 47538
H2O_NCU_TRAFFIC_BYTES = 2055e6         # h2o_compact_kernel, 64-request eviction workload
OMNIKV_NCU_TRAFFIC_BYTES = 209e6       # token_decode_kernel, 24-request selection-reuse workload


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while running."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples = []
        self._stop = threading.Event()
        self._thread = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_sm = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), sm, reasons))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.ok:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self, t0: float, t1: float):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": ["unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = None
        if not inside:                       # timed region shorter than one sampling period
            inside = sorted(self.samples, key=lambda s: abs(s[0] - 0.5 * (t0 + t1)))[:3]
            note = "nearest_samples"
        names = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        bits = 0
        for s in inside:
            bits |= int(s[2])
        reasons = [n for b, n in names.items() if bits & b]
        out = {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.max_sm,
               "reasons": reasons, "samples": len(inside)}
        if note:
            out["note"] = note
        return out


# ------------------------------------------------------------------ workload accounting
def algorithmic_bytes(w, sel_cnt, h2o: bool):
    """Bytes the method must move per step (per layer): summaries of every present page,
    K and V of the selected pages, q, out, lse (+ the H2O read-modify-write)."""
    pt = w.page_table.cpu().numpy()
    sl = w.seq_lens.cpu().numpy()
    n_r = (sl + 15) // 16
    present = sum(int((pt[r, :n_r[r]] >= 0).sum()) for r in range(w.B))
    meta = present * w.H_kv * 2 * w.D * 2
    k_eff = int(sel_cnt.sum().item())
    kv = k_eff * 16 * w.D * 2 * 2
    q = w.B * w.H_q * w.D * 2
    outlse = w.B * w.H_q * (4 * w.D + 4)
    accum = 0
    if h2o:
        accum = 2 * 4 * 16 * k_eff          # upper bound: every slot of every selected page
    return dict(meta=meta, kv=kv, q=q, outlse=outlse, accum=accum,
                select_call=meta + q, decode_kernel=kv + q + outlse,
                total=meta + kv + q + outlse + accum, present_pages=present, selected_pages=k_eff)


def checksums(w):
    """64-bit sums of the raw bits of the seeded inputs (reproducibility record, not arithmetic of the method)."""
    def s64(t):
        v = t.contiguous().view(torch.int32) if t.element_size() * t.numel() % 4 == 0 else t.contiguous().view(torch.int16)
        return "%016x" % (int(v.sum(dtype=torch.int64).item()) & 0xFFFFFFFFFFFFFFFF)
    return {"q": s64(w.q), "k_cache": s64(w.k_cache), "v_cache": s64(w.v_cache),
            "page_table": s64(w.page_table), "seq_lens": s64(w.seq_lens)}


def make_layers(config: int, device, n_layers: int, rank: int, batch: int = 0, instance: int = 0, hi: int = 0):
    """The layers of one instance of a config.  Structure (lengths, page table) is the same for every layer
    and instance; q/K/V values differ (seeded by layer index; other instances and ranks use other layer seeds)."""
    fn = wl.CONFIGS[config]
    if batch or hi:
        base = fn
        kw = dict(B=batch) if batch else {}
        if hi:
            kw["hi"] = hi
        fn = lambda device, layer=0: base(device, layer=layer, **kw)
    layers = []
    first = None
    for l in range(n_layers):
        w = fn(device, layer=l + 100 * rank + 1000 * instance)
        if first is None:
            first = w
        else:                                 # the block table is per request, shared by all layers
            w.page_table, w.seq_lens = first.page_table, first.seq_lens
        layers.append(w)
    return layers


# ------------------------------------------------------------------ CPU oracle timing
def _omp_set_threads(n: int):
    """Thread count of the oracle's OpenMP loops for the following calls (a libgomp call, not oracle code)."""
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except Exception:
        return False


def oracle_step_time(w, meta_bits, threads=None, min_runs=3, budget_s=20.0):
    """The oracle, as it stands, on the WHOLE batch of ``w`` (one layer): seconds per decode step, best of
    >= min_runs.  ``meta_bits``: the page summaries (the rebuild after prefill is set-up for both sides)."""
    import oracle
    w_cpu = w.to("cpu")
    q, k, v = wl.bf16_bits(w_cpu.q), wl.bf16_bits(w_cpu.k_cache), wl.bf16_bits(w_cpu.v_cache)
    pt, sl = w_cpu.page_table.numpy(), w_cpu.seq_lens.numpy()
    u = None if w_cpu.score_accum is None else w_cpu.score_accum.numpy().astype(np.float64)
    cores = oracle.num_threads()
    if threads is not None and _omp_set_threads(threads):
        cores = threads
    times = []
    t_begin = time.perf_counter()
    while len(times) < min_runs or (time.perf_counter() - t_begin < budget_s and len(times) < 10):
        t0 = time.perf_counter()
        oracle.decode_step(q, k, v, pt, sl, w_cpu.budget, meta=meta_bits, u_accum=None if u is None else u.copy())
        times.append(time.perf_counter() - t0)
    if threads is not None:
        _omp_set_threads(oracle.num_threads())
    return min(times), len(times), cores


# ------------------------------------------------------------------ one config on one rank
class Instance:
    """One independent copy of a config's layers with its states, H2O accumulators and the graph of its step."""

    def __init__(self, binding, config, dev, n_layers, rank, batch, index, dense_layers=0, use_graph=True, hi=0):
        self.layers = make_layers(config, dev, n_layers, rank, batch, index, hi)
        w0 = self.layers[0]
        self.h2o = w0.score_accum is not None
        self.dense_layers = dense_layers
        self.states = []
        shared = {}                            # layers with the same shape share one workspace, as an engine would
        for l, w in enumerate(self.layers):
            k_max = w0.max_pages if l < dense_layers else None
            st = binding.DecodeState(w, k_max=k_max, workspace=shared.get(k_max))
            shared.setdefault(k_max, st.workspace)
            self.states.append(st)
        self.accums = [w.score_accum.clone() if self.h2o else None for w in self.layers]
        for st in self.states:
            st.rebuild_meta()
        torch.cuda.synchronize()
        self.graph = None
        if use_graph:
            s = torch.cuda.Stream()
            s.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s):
                self.step()
            torch.cuda.current_stream().wait_stream(s)
            torch.cuda.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph):
                self.step()
        self.step()
        torch.cuda.synchronize()
        for st in self.states:
            if st.status() != 0:
                raise SystemExit("device status word not clean")

    def step(self):
        for l, (st, u) in enumerate(zip(self.states, self.accums)):
            if l < self.dense_layers:
                st.step(score_accum=u, budget=16 * st.w.max_pages)
            else:
                st.step(score_accum=u)

    def run(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.step()


class Flusher:
    """Evicts the step's data from L2: a 252 MiB write, then a 252 MiB read of another buffer, so that the
    lines the timed step displaces are clean (displacing the write's dirty lines would charge the step one
    write-back per byte it reads)."""

    def __init__(self, dev):
        self.buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        self.src = torch.zeros(2 * L2_BYTES // 4, dtype=torch.int32, device=dev)
        self.sink = torch.zeros(1, dtype=torch.int32, device=dev)
        self.i = 0

    def __call__(self):
        self.i += 1
        self.buf.fill_(self.i & 0xFF)
        self.sink.copy_(self.src.max().reshape(1))


def chained_graph(insts):
    """One CUDA graph that runs the steps of ``insts`` one after the other; returns its replay function."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for i in insts:
            i.step()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in insts:
            i.step()
    return g.replay


def timed_windows(run_one, K, barrier, world, dev, flusher=None):
    """K timed steps in up to three windows (32 untimed replays in front of each); returns (ms per step,
    per-window ms per step, wall-clock interval)."""
    n_win = 3 if K >= 96 else 1
    sizes = [K // n_win] * n_win
    sizes[-1] += K - sum(sizes)
    per_window = []
    t_wall0 = time.perf_counter()
    for n in sizes:
        for _ in range(WINDOW_WARMUP):
            run_one()
        barrier()
        if flusher is not None:
            starts = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
            ends = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
            for i in range(n):
                flusher()
                starts[i].record()
                run_one()
                ends[i].record()
            barrier()
            ms = sum(a.elapsed_time(b) for a, b in zip(starts, ends))
        else:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                run_one()
            e1.record()
            barrier()
            ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
            ms = float(t.item())
        per_window.append(ms / n)
    t_wall1 = time.perf_counter()
    total = sum(m * n for m, n in zip(per_window, sizes))
    return total / K, per_window, (t_wall0, t_wall1)


class E2E:
    """The step driven from HOST buffers the way a serving loop drives the library: per step one pinned
    block per layer goes up (q; with layer 0 also the lengths and the page-table entries that changed -
    one per request: the entry of its newest page), the step runs, out + lse come back into pinned
    memory, and the host waits for them.  Uploads, steps and downloads of consecutive layers overlap
    (three streams inside one graph)."""

    def __init__(self, inst: Instance, dev, use_graph=True):
        self.inst = inst
        w0 = inst.layers[0]
        B = w0.B
        sl = w0.seq_lens.cpu()
        pt = w0.page_table.cpu()
        col = ((sl.to(torch.int64) - 1).clamp(min=0)) // 16
        flat = torch.arange(B, dtype=torch.int64) * w0.max_pages + col
        newest = pt.view(-1)[flat].clone()
        self.up_host, self.up_dev, self.views = [], [], []
        self.dn_host, self.dn_dev = [], []
        self.states = []
        import copy
        for l, (w, st) in enumerate(zip(inst.layers, inst.states)):
            tensors = [w.q] + ([w.seq_lens, flat.to(dev), newest.to(dev)] if l == 0 else [])
            hb, hv = self._packed(tensors, "cpu", True)
            db, dv = self._packed(tensors, dev, False)
            for src, h_, d_ in zip(tensors, hv, dv):
                h_.copy_(src)
                d_.copy_(src)
            ob, ov = self._packed([st.out, st.lse], dev, False)
            hob, _ = self._packed([st.out, st.lse], "cpu", True)
            st2 = copy.copy(st)               # same params, workspace, summaries and selection buffers
            st2.w = dataclasses.replace(w, q=dv[0], seq_lens=(dv[1] if l == 0 else self.states[0].w.seq_lens))
            st2.out, st2.lse = ov
            self.states.append(st2)
            self.up_host.append(hb); self.up_dev.append(db); self.views.append(dv)
            self.dn_host.append(hob); self.dn_dev.append(ob)
        self.h2d = sum(b.numel() for b in self.up_host)
        self.d2h = sum(b.numel() for b in self.dn_host)
        self.s_up, self.s_dn = torch.cuda.Stream(), torch.cuda.Stream()
        self.graph = None
        if use_graph:
            s = torch.cuda.Stream()
            s.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s):
                self.body()
            torch.cuda.current_stream().wait_stream(s)
            torch.cuda.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph):
                self.body()

    @staticmethod
    def _packed(tensors, device, pin):
        """One byte block holding the tensors back to back (16-byte aligned); returns (block, views)."""
        offs, total = [], 0
        for t in tensors:
            offs.append(total)
            total += (t.numel() * t.element_size() + 15) // 16 * 16
        block = torch.empty(total, dtype=torch.uint8, device=device)
        if pin:
            block = block.pin_memory()
        views = [block[o:o + t.numel() * t.element_size()].view(t.dtype).view(t.shape) for o, t in zip(offs, tensors)]
        return block, views

    def body(self):
        main = torch.cuda.current_stream()
        inst = self.inst
        self.s_up.wait_stream(main)
        ups, dones = [], []
        with torch.cuda.stream(self.s_up):
            for hb, db in zip(self.up_host, self.up_dev):
                db.copy_(hb, non_blocking=True)
                ev = torch.cuda.Event()
                ev.record()
                ups.append(ev)
        for l, (st2, u) in enumerate(zip(self.states, inst.accums)):
            main.wait_event(ups[l])
            if l == 0:                       # the page-table entries that changed since the last step
                pt = inst.layers[0].page_table
                pt.view(-1).index_copy_(0, self.views[0][2], self.views[0][3])
            if l < inst.dense_layers:
                st2.step(score_accum=u, budget=16 * st2.w.max_pages)
            else:
                st2.step(score_accum=u)
            ev = torch.cuda.Event()
            ev.record()
            dones.append(ev)
        with torch.cuda.stream(self.s_dn):
            for l, (ob, hob) in enumerate(zip(self.dn_dev, self.dn_host)):
                self.s_dn.wait_event(dones[l])
                hob.copy_(ob, non_blocking=True)
        main.wait_stream(self.s_dn)
        main.wait_stream(self.s_up)

    def step(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.body()
        torch.cuda.synchronize()              # the host needs the result before the next step


def gather_ceilings(binding, inst: Instance, dev, iters=20):
    """Read-only gathers with the access pattern and pipeline shape of the two streaming kernels on the
    very pages layer 0 reads (se_probe_gather): what the memory system allows for those patterns."""
    w, st = inst.layers[0], inst.states[0]
    pt = w.page_table.to(torch.int64)
    n_r = (w.seq_lens.to(torch.int64) + 15) // 16
    cols = torch.arange(w.max_pages, device=dev)[None, :]
    present = (cols < n_r[:, None]) & (pt >= 0)
    heads = torch.arange(w.H_kv, device=dev, dtype=torch.int64)
    # summaries: (request, kv-head, page) order, piece = pid*H_kv + h
    pieces = []
    for r in range(w.B):
        pid = pt[r][present[r]]
        pieces.append((pid[None, :] * w.H_kv + heads[:, None]).reshape(-1))
    meta_idx = torch.cat(pieces).to(torch.int32).contiguous()
    # selected pages: K page and V page of the same index next to each other
    sel = st.sel_idx.to(torch.int64)
    cnt = st.sel_cnt
    ok = torch.arange(st.k_max, device=dev)[None, None, :] < cnt[:, :, None]
    rr = torch.arange(w.B, device=dev)[:, None, None].expand_as(sel)
    hh = heads[None, :, None].expand_as(sel)
    pid = pt[rr[ok], sel[ok]]
    kv_idx = (pid * w.H_kv + hh[ok]).to(torch.int32)
    kv_idx = torch.stack([kv_idx, kv_idx], dim=1).reshape(-1).contiguous()
    out = {}

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters * 1e3

    row = 2 * w.D * 2
    us = timed(lambda: binding.se_probe_gather(st.meta, meta_idx, row, 16, 2, 4, 3))
    out["summaries_%dB" % row] = {"us": us, "bytes": int(meta_idx.numel()) * row, "gbs": int(meta_idx.numel()) * row / us / 1e3,
                                  "shape": "16 pieces x 2 stages x 4 warps x 3 CTAs/SM"}
    page = 16 * w.D * 2
    us = timed(lambda: binding.se_probe_gather(w.k_cache, kv_idx, page, 2, 5, 4, 1, base1=w.v_cache))
    out["pages_%dB" % page] = {"us": us, "bytes": int(kv_idx.numel()) * page, "gbs": int(kv_idx.numel()) * page / us / 1e3,
                               "shape": "K+V page x 5 stages x 4 warps x 1 CTA/SM"}
    return out


def run_config(binding, config, dev, args, rank, world, barrier, full: bool, K: int):
    """Times one config on this rank.  ``full``: also the per-call times, rooflines, the end-to-end number and
    the gather ceilings; otherwise a short record for ``other_configs``."""
    n_layers = args.layers if (full and args.layers) else (28 if config == 5 else 1)
    batch = args.batch if full else 0
    use_graph = not args.no_graph
    dense = args.dense_layers if (full or config == 5) else 0
    hi = args.hi if full else 0
    inst0 = Instance(binding, config, dev, n_layers, rank, batch, 0, dense_layers=dense, use_graph=use_graph, hi=hi)
    layers, states = inst0.layers, inst0.states
    h2o = inst0.h2o
    bytes_l = [algorithmic_bytes(st.w, st.sel_cnt, h2o) for st in states]
    total_bytes = sum(b["total"] for b in bytes_l)
    # cold L2: by size, by rotation over R independent instances (R steps touch >= 4 x L2), or by a flush
    mode, instances, flusher = "stream", [inst0], None
    if total_bytes < 2 * L2_BYTES:
        R = -(-4 * L2_BYTES // total_bytes)
        if R <= 8:
            mode = "rotate"
            instances += [Instance(binding, config, dev, n_layers, rank, batch, i, dense_layers=dense, use_graph=use_graph, hi=hi)
                          for i in range(1, R)]
        else:
            mode = "flush"
            flusher = Flusher(dev)
    turn = [0]

    def run_one():
        instances[turn[0] % len(instances)].run()
        turn[0] += 1

    # Steps of a few tens of microseconds: a serving engine replays the layers of a model step as ONE graph,
    # so the steps of the R instances are chained into one graph of `chain` steps (a replay per step would
    # add the graph-launch gap, several microseconds, to every step).
    chain, run_chain = 1, None
    if mode == "rotate" and use_graph:
        chain = len(instances) * max(1, 8 // len(instances))
        if K % chain == 0:
            run_chain = chained_graph([instances[i % len(instances)] for i in range(chain)])
        else:
            chain = 1

    sampler = ClockSampler(dev.index)
    sampler.start()
    for _ in range(max(args.warmup, 3)):       # the discarded run
        run_one()
    barrier()
    if run_chain is not None:
        ms_chain, windows, (t0, t1) = timed_windows(run_chain, K // chain, barrier, world, dev, None)
        ms_per_step, windows = ms_chain / chain, [m / chain for m in windows]
    else:
        ms_per_step, windows, (t0, t1) = timed_windows(run_one, K, barrier, world, dev, flusher)
    clocks = sampler.summary(t0, t1)
    peak, peak_kind = measured_peak()
    step_gbs = total_bytes / (ms_per_step * 1e-3) / 1e9
    w0 = layers[0]
    rec = {
        "value": ms_per_step * 1e3, "unit": "us", "steps": K, "windows_us": [m * 1e3 for m in windows],
        "config": {
            "workload": w0.name, "config_id": config, "layers": n_layers, "B": w0.B, "H_q": w0.H_q, "H_kv": w0.H_kv,
            "D": w0.D, "page_size": 16, "budget_tokens": w0.budget, "storage_dtype": "bf16",
            "present_pages": bytes_l[0]["present_pages"], "selected_pages": bytes_l[0]["selected_pages"],
            "h2o_epilogue": h2o, "cuda_graph": use_graph, "dense_layers": dense,
            "l2": {"stream": "inputs larger than L2 (%.0f MB touched per step)" % (total_bytes / 1e6),
                   "rotate": "%d independent instances in turn (%.0f MB per step, %.0f MB before an instance is touched "
                             "again), %d steps chained per graph replay" % (len(instances), total_bytes / 1e6,
                                                                             len(instances) * total_bytes / 1e6, chain),
                   "flush": "flushed before every step: a %d MiB write, then a %d MiB read (leaves clean lines); the "
                            "step then pays its launch latency inside the timed region" % (2 * L2_BYTES >> 20, 2 * L2_BYTES >> 20)}[mode],
            "protocol": "1 discarded run, %d window(s) of 32 untimed + %s timed replays" % (len(windows), "/".join(str(int(round(K / len(windows)))) for _ in windows)),
            "parallelism": "1 GPU" if world == 1 else "%d replicas, no collective" % world,
            "global_batch": w0.B * world,
        },
        "algorithmic_bytes_per_step": total_bytes,
        "achieved_gbs": step_gbs * world,
        "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
        "frac_of_measured_copy": step_gbs / peak,
        "launches_per_step": sum(binding.se_decode_step_launches(st.p, 16 * st.w.max_pages if l < dense else st.w.budget, h2o)
                                 for l, st in enumerate(states)),
        "clocks": clocks,
    }
    # warm L2 (same instance back to back) where the step fits in L2, and the flush-based latency of one step
    if mode != "stream":
        warm = chained_graph([inst0] * 8) if use_graph else inst0.run
        per = 8 if use_graph else 1
        for _ in range(5):
            warm()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = max(5, min(K, 200) // per)
        a.record()
        for _ in range(n):
            warm()
        b.record()
        torch.cuda.synchronize()
        rec["l2_warm_us"] = a.elapsed_time(b) / (n * per) * 1e3
        del warm
        fl = flusher or Flusher(dev)
        tot = 0.0
        n = 30
        for _ in range(n):
            fl()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); inst0.run(); b.record()
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        rec["single_step_after_flush_us"] = tot / n * 1e3
        del fl

    # ---- end to end
    e2e = E2E(inst0, dev, use_graph)
    for _ in range(3):
        e2e.step()
    e2e_iters = max(10, min(K, 200 if n_layers == 1 else 30))
    others = [E2E(i, dev, use_graph) for i in instances[1:]] if mode == "rotate" else []
    ring = [e2e] + others
    barrier()
    tot_ms = 0.0
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if flusher is None:
        a.record()
        for i in range(e2e_iters):
            ring[i % len(ring)].step()
        b.record()
        barrier()
        tot_ms = a.elapsed_time(b)
    else:
        for i in range(e2e_iters):
            flusher()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); e2e.step(); b.record()
            torch.cuda.synchronize()
            tot_ms += a.elapsed_time(b)
    e2e_ms = tot_ms / e2e_iters
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        e2e_ms = float(t.item())
    rec["e2e"] = {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": e2e.h2d, "d2h_bytes_per_step": e2e.d2h,
                  "what": "pinned q (+ lengths and the changed page-table entries) up, step, out + lse down into pinned "
                          "memory, host sync; copies of consecutive layers overlap the steps"}
    del others, ring
    sampler.stop()

    if full:
        rec.update(per_call_and_rooflines(binding, inst0, dev, bytes_l[0], flusher if mode == "flush" else None, K, peak, peak_kind))
        rec["config"]["checksums_layer0"] = checksums(w0)
    rec["_inst0"] = inst0
    return rec


def per_call_and_rooflines(binding, inst, dev, b0, flusher, K, peak, peak_kind):
    """Every entry point timed on its own (same stream, CUDA events, each call in its own loop) and the
    roofline record of the two streaming kernels."""
    st0, u0 = inst.states[0], inst.accums[0]
    w0 = inst.layers[0]

    def time_call(fn, iters):
        for _ in range(3):
            fn()
        if flusher is not None:
            tot = 0.0
            for i in range(iters):
                flusher()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                tot += a.elapsed_time(b)
            return tot / iters * 1e3
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters * 1e3

    iters = max(10, min(K, 200))
    call_us = {
        "se_meta_update": time_call(st0.update_meta, iters),
        "se_page_select": time_call(st0.select, iters),
        "se_page_select_scores": time_call(lambda: st0.select(entry="se_page_select_scores"), iters),
        "se_page_select_topk": time_call(lambda: st0.select(entry="se_page_select_topk"), iters),
        "se_page_select_fused": time_call(st0.select_fused, iters),
        "se_sparse_decode": time_call(lambda: st0.decode(u0), iters),
        "se_sparse_decode_splits": time_call(lambda: st0.decode(u0, entry="se_sparse_decode_splits"), iters),
        "se_combine": time_call(lambda: st0.decode(u0, entry="se_combine"), iters),
        "se_decode_step": time_call(lambda: st0.step(u0), iters),
    }
    ceil = gather_ceilings(binding, inst, dev)
    c_meta = next(v for k, v in ceil.items() if k.startswith("summaries"))
    c_kv = next(v for k, v in ceil.items() if k.startswith("pages"))
    dec_gbs = b0["decode_kernel"] / (call_us["se_sparse_decode_splits"] * 1e-6) / 1e9
    score_gbs = b0["select_call"] / (call_us["se_page_select_scores"] * 1e-6) / 1e9
    rl_decode = {"bound": "hbm", "kernel": "attention kernel (se_sparse_decode_splits)", "achieved": dec_gbs,
                 "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": dec_gbs / peak,
                 "traffic": NCU_TRAFFIC_BYTES.get(w0.name), "algorithmic_bytes": b0["decode_kernel"],
                 "us": call_us["se_sparse_decode_splits"], "gather_ceiling_gbs": c_kv["gbs"],
                 "frac_of_gather_ceiling": dec_gbs / c_kv["gbs"]}
    rl_score = {"bound": "hbm", "kernel": "score_kernel (se_page_select_scores)", "achieved": score_gbs,
                "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": score_gbs / peak,
                "traffic": NCU_TRAFFIC_BYTES_SCORE.get(w0.name), "algorithmic_bytes": b0["select_call"],
                "us": call_us["se_page_select_scores"], "gather_ceiling_gbs": c_meta["gbs"],
                "frac_of_gather_ceiling": score_gbs / c_meta["gbs"]}
    # the dominant kernel is whichever of the two streaming kernels takes longer on this workload
    rl_main, rl_other = (rl_score, rl_decode) if rl_score["us"] >= rl_decode["us"] else (rl_decode, rl_score)
    return {"calls_us": call_us, "roofline": rl_main, "roofline_second_kernel": rl_other, "gather_ceiling": ceil}


def spawn_ranks(args):
    """bench.py --gpus N without a rank environment: start the N ranks ourselves, one per GPU."""
    port = 29500 + (os.getpid() % 2000)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


# ------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=768, help="timed steps (default 768 = 3 windows of 256)")
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--config", type=int, default=3, choices=sorted(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="layers per step (default 1; 28 for config 5)")
    ap.add_argument("--dense-layers", type=int, default=0,
                    help="the first this many layers attend every page (budget >= context), the others select under "
                         "the budget (the paper's per-layer policy); all in the same graph")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=0,
                    help="override the number of requests (configs 3-5; for small profiling captures)")
    ap.add_argument("--hi", type=int, default=0,
                    help="override the longest context of configs 3 and 5 (for small profiling captures)")
    ap.add_argument("--no-graph", action="store_true", help="launch the calls directly instead of a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the short runs of the other configs")
    ap.add_argument("--workload", default="decode", choices=["decode", "h2o_evict", "omnikv_reuse"],
                    help="decode = the sparse decode step (the headline); h2o_evict = one H2O eviction "
                         "(retained set + in-place compaction) of 64 requests, 5120 -> 4096 tokens; "
                         "omnikv_reuse = one observation layer (full attention + token selection) and four "
                         "sparse layers reusing its 2048+32 tokens, 24 requests of 32768 tokens")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.gpus > 1 and "RANK" not in os.environ and args.impl == "ours" and args.workload == "decode":
        spawn_ranks(args)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.workload in ("h2o_evict", "omnikv_reuse"):
        if rank == 0:                        # these steps have no multi-GPU leg of their own
            (run_h2o_evict if args.workload == "h2o_evict" else run_omnikv)(args, local_rank)
        return
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2609_39068_b200 import binding
    binding.load()

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    K = args.steps
    rec = run_config(binding, args.config, dev, args, rank, world, barrier, True, K)
    inst0 = rec.pop("_inst0")
    n_layers = rec["config"]["layers"]

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, runs, cores = oracle_step_time(inst0.layers[0], wl.bf16_bits(inst0.states[0].meta))
        cpu_baseline = dict(value=sec * n_layers * 1e6, unit="us", cores=cores, kind="oracle",
                            sample="the whole batch (%d requests) of layer 0, fp64 C oracle with OpenMP over (request, "
                                   "kv-head), best of %d runs = %.1f ms%s" % (inst0.layers[0].B, runs, sec * 1e3,
                                   "; x%d layers" % n_layers if n_layers > 1 else ""),
                            sample_seconds=sec)
    del inst0
    torch.cuda.empty_cache()

    other = None
    if rank == 0 and world == 1 and not args.no_other_configs and not args.batch and not args.hi:
        other = {}
        for c in sorted(wl.CONFIGS):
            if c == args.config:
                continue
            r = run_config(binding, c, dev, args, rank, world, barrier, False, 96 if c != 5 else 12)
            i0 = r.pop("_inst0")
            if c in (1, 2) and not args.no_cpu_baseline:
                meta_bits = wl.bf16_bits(i0.states[0].meta)
                sec, runs, cores = oracle_step_time(i0.layers[0], meta_bits, budget_s=3.0)
                sec1, runs1, _ = oracle_step_time(i0.layers[0], meta_bits, threads=1, budget_s=3.0)
                r["cpu_baseline"] = {"value": sec * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
                                     "one_thread_us": sec1 * 1e6, "sample": "whole batch, best of %d / %d runs" % (runs, runs1)}
            other["config%d" % c] = r
            del i0
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": rec["value"], "unit": "us", "n_gpus": world,
            "steps": K, "warmup": args.warmup, "ms_per_step": rec["value"] / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
        }
        line.update({k: v for k, v in rec.items() if k not in ("value", "unit", "steps")})
        line["gpu_launches"] = rec["launches_per_step"] * K
        line["cpu_baseline"] = cpu_baseline
        if other is not None:
            line["other_configs"] = other
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def h2o_oracle_time(w, budget, recent, n_sample=8):
    """The oracle's retained set + compaction on a few requests, scaled to the batch by request count."""
    import oracle
    rows = list(range(0, w.B, max(1, w.B // n_sample)))[:n_sample]
    sub = wl.sub_workload(w, rows, "cpu")
    k, v = wl.bf16_bits(sub.k_cache), wl.bf16_bits(sub.v_cache)
    u = sub.score_accum.numpy().astype(np.float64)
    pt, sl = sub.page_table.numpy(), sub.seq_lens.numpy()
    times = []
    for _ in range(3):
        t0 = time.perf_counter()
        idx, cnt = oracle.h2o_retain(u, pt, sl, budget, recent)
        oracle.h2o_compact(k, v, u, pt, idx, cnt)
        times.append(time.perf_counter() - t0)
    best, scale = min(times), w.B / float(len(rows))
    return dict(value=best * scale * 1e6, unit="us", cores=oracle.num_threads(), kind="oracle",
                sample="%d of %d requests, retained set (OpenMP over pairs) + compaction (one thread), best of 3 "
                       "= %.1f ms, scaled x%.1f by request count" % (len(rows), w.B, best * 1e3, scale))


def run_h2o_evict(args, local_rank):
    """One H2O eviction step: se_h2o_retain + se_h2o_compact on 64 requests that are 1024 tokens over
    their 4096-token budget (recent ratio 0.2).  The scores are restored (untimed) before every step,
    so every step evicts the same tokens; K/V values do not influence the work."""
    budget, recent = 4096, 819
    if args.impl == "reference":
        dev = "cuda" if torch.cuda.is_available() else "cpu"
        w = wl.h2o_evict_workload(dev) if dev == "cuda" else wl.h2o_evict_workload(dev, B=8)
        cb = h2o_oracle_time(w, budget, recent)
        print(json.dumps({
            "impl": "reference", "metric": "h2o_evict_us_per_step", "value": cb["value"], "unit": "us",
            "n_gpus": args.gpus, "steps": 3, "warmup": 0, "ms_per_step": cb["value"] / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name}, "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    from paper_2609_39068_b200 import binding
    binding.load()
    w = wl.h2o_evict_workload(dev, B=args.batch or 64)
    p = binding.make_params(w.B, w.H_q, w.H_kv, w.D, w.max_pages, w.num_phys_pages, 1)
    ws = binding.alloc_workspace(p, dev)
    keep_idx = torch.empty((w.B, w.H_kv, budget), dtype=torch.int32, device=dev)
    keep_cnt = torch.empty((w.B, w.H_kv), dtype=torch.int32, device=dev)
    new_lens = torch.empty((w.B,), dtype=torch.int32, device=dev)
    u0 = w.score_accum.clone()
    lens_pin = w.seq_lens.cpu().pin_memory()
    out_pin = torch.empty((w.B,), dtype=torch.int32).pin_memory()

    def retain():
        binding.se_h2o_retain(p, w.score_accum, w.page_table, w.seq_lens, budget, recent, keep_idx, keep_cnt, ws)

    def compact():
        binding.se_h2o_compact(p, w.k_cache, w.v_cache, w.score_accum, w.page_table, keep_idx, keep_cnt,
                               new_lens, ws)

    def timed(fns, iters, e2e=False):
        tot = 0.0
        for _ in range(iters):
            w.score_accum.copy_(u0)                      # untimed: same eviction every step
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if e2e:
                w.seq_lens.copy_(lens_pin, non_blocking=True)
            for fn in fns:
                fn()
            if e2e:
                out_pin.copy_(new_lens, non_blocking=True)
            b.record()
            torch.cuda.synchronize()
            tot += a.elapsed_time(b)
        return tot / iters * 1e3

    K = min(args.steps, 200)
    sampler = ClockSampler(local_rank)
    sampler.start()
    timed([retain, compact], args.warmup)
    t0 = time.perf_counter()
    step_us = timed([retain, compact], K)
    t1 = time.perf_counter()
    w.score_accum.copy_(u0)
    retain()
    retain_us = timed([retain], 50)
    compact_us = timed([compact], 50)                    # keep_idx of the step above, scores restored each time
    e2e_us = timed([retain, compact], 50, e2e=True)
    sampler.stop()
    status = binding.se_last_device_status(ws)
    if status:
        raise SystemExit("device status %d" % status)
    # algorithmic bytes: every destination page that holds a moved token is read and written once
    ki = keep_idx.cpu().numpy().reshape(-1, budget)
    moved_tok = ki != np.arange(budget)[None, :]
    moved_pages = int(moved_tok.reshape(ki.shape[0], budget // 16, 16).any(axis=2).sum())
    row_bytes = 2 * w.D * 2 + 4                          # K row + V row + score
    compact_bytes = moved_pages * 16 * row_bytes * 2 + ki.size * 4
    retain_bytes = int(w.seq_lens.sum().item()) * w.H_kv * 4 + ki.size * 4
    peak, peak_kind = measured_peak()
    cb = None if args.no_cpu_baseline else h2o_oracle_time(w, budget, recent)
    gbs = compact_bytes / (compact_us * 1e-6) / 1e9
    print(json.dumps({
        "metric": "h2o_evict_us_per_step", "value": step_us, "unit": "us", "n_gpus": 1, "steps": K,
        "warmup": args.warmup, "ms_per_step": step_us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H_kv": w.H_kv, "D": w.D, "cached_tokens": 5120,
                   "budget_tokens": budget, "recent_tokens": recent, "moved_pages": moved_pages,
                   "l2": "inputs larger than L2 (%d MB moved per step)" % (compact_bytes // 10**6)},
        "calls_us": {"se_h2o_retain": retain_us, "se_h2o_compact": compact_us},
        "algorithmic_bytes": {"se_h2o_retain": retain_bytes, "se_h2o_compact": compact_bytes},
        "roofline": {"bound": "hbm", "kernel": "h2o_compact_kernel (se_h2o_compact)", "achieved": gbs, "peak": peak,
                     "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": gbs / peak,
                     "traffic": H2O_NCU_TRAFFIC_BYTES if w.B == 64 else None,
                     "algorithmic_bytes": compact_bytes},
        "clocks": sampler.summary(t0, t1),
        "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": w.B * 4, "d2h_bytes_per_step": w.B * 4},
        "gpu_launches": 2 * K, "cpu_baseline": cb}))


def omnikv_oracle_time(layers, budget, recent, n_sample=2):
    """The oracle's observation layer (scores, full attention, token top-k) + reuse layers on a few requests."""
    import oracle
    w0 = layers[0]
    rows = list(range(0, w0.B, max(1, w0.B // n_sample)))[:n_sample]
    subs = [wl.sub_workload(w, rows, "cpu") for w in layers]
    a0 = subs[0]
    pt, sl = a0.page_table.numpy(), a0.seq_lens.numpy()
    n_pages = (sl + 15) // 16
    sel = np.full((a0.B, a0.H_kv, a0.max_pages), -1, np.int32)
    scnt = np.zeros((a0.B, a0.H_kv), np.int32)
    for r in range(a0.B):
        sel[r, :, :n_pages[r]] = np.arange(n_pages[r])
        scnt[r, :] = n_pages[r]
    bits = [(wl.bf16_bits(x.q), wl.bf16_bits(x.k_cache), wl.bf16_bits(x.v_cache)) for x in subs]
    t0 = time.perf_counter()
    s, present = oracle.token_scores(bits[0][0], bits[0][1], pt, sl)
    oracle.attend(bits[0][0], bits[0][1], bits[0][2], pt, sl, sel, scnt)
    idx, cnt, _ = oracle.token_topk(s, present, sl, budget, recent)
    for q, k, v in bits[1:]:
        oracle.token_attend(q, k, v, pt, sl, idx, cnt)
    dt = time.perf_counter() - t0
    scale = w0.B / float(len(rows))
    return dict(value=dt * scale * 1e6, unit="us", cores=oracle.num_threads(), kind="oracle",
                sample="%d of %d requests, one run = %.2f s, scaled x%.1f by request count" % (len(rows), w0.B, dt, scale))


def run_omnikv(args, local_rank):
    """Selection reuse across layers: layer 0 = observation layer (full attention that also scores every
    token, then the token top-k), layers 1-4 = sparse layers attending the 2048 selected + 32 recent
    tokens of their own caches.  One step = se_observe_decode + se_token_select + 4 x se_token_decode."""
    budget, recent, n_sparse = 2048, 32, 4
    if not torch.cuda.is_available():
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the selection-reuse workload is generated on the GPU"}))
            return
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B = args.batch or 24
    layers = [wl.omnikv_workload(dev, layer=l, B=B) for l in range(1 + n_sparse)]
    if args.impl == "reference":
        cb = omnikv_oracle_time(layers, budget, recent)
        print(json.dumps({
            "impl": "reference", "metric": "omnikv_reuse_us_per_step", "value": cb["value"], "unit": "us",
            "n_gpus": args.gpus, "steps": 1, "warmup": 0, "ms_per_step": cb["value"] / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": layers[0].name}, "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return
    from paper_2609_39068_b200 import binding
    binding.load()
    w0 = layers[0]
    obs = binding.DecodeState(w0, k_max=w0.max_pages)
    obs.w = wl.Workload(**{**w0.__dict__, "budget": 16 * w0.max_pages})
    obs.rebuild_meta()
    obs.select()                                   # full attention: every present page, selected once
    n_out = budget + recent
    keys = torch.zeros((B, 16 * w0.max_pages), dtype=torch.int32, device=dev)
    tok_idx = torch.empty((B, n_out), dtype=torch.int32, device=dev)
    tok_cnt = torch.empty((B,), dtype=torch.int32, device=dev)
    p_tok = binding.make_params(B, w0.H_q, w0.H_kv, w0.D, w0.max_pages, w0.num_phys_pages, (n_out + 15) // 16)
    ws_tok = binding.alloc_workspace(p_tok, dev)
    outs = [(torch.empty((B, w0.H_q, w0.D), dtype=torch.float32, device=dev),
             torch.empty((B, w0.H_q), dtype=torch.float32, device=dev)) for _ in range(n_sparse)]

    def observe():
        binding.se_observe_decode(obs.p, w0.q, w0.k_cache, w0.v_cache, w0.page_table, w0.seq_lens, obs.sel_idx,
                                  obs.sel_cnt, obs.out, obs.lse, keys, obs.workspace)

    def select():
        binding.se_token_select(obs.p, keys, w0.seq_lens, budget, recent, tok_idx, tok_cnt, obs.workspace)

    def reuse(i):
        w = layers[1 + i]
        binding.se_token_decode(p_tok, w.q, w.k_cache, w.v_cache, w.page_table, w.seq_lens, tok_idx, tok_cnt,
                                outs[i][0], outs[i][1], ws_tok)

    def step():
        observe()
        select()
        for i in range(n_sparse):
            reuse(i)

    q_pin = [w.q.cpu().pin_memory() for w in layers]
    o_pin = [torch.empty(o.shape, dtype=torch.float32).pin_memory() for o, _ in outs]

    def step_e2e():
        for w, qp in zip(layers, q_pin):
            w.q.copy_(qp, non_blocking=True)
        step()
        for (o, _), op in zip(outs, o_pin):
            op.copy_(o, non_blocking=True)

    def timed(fn, iters):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters * 1e3

    K = min(args.steps, 100)
    sampler = ClockSampler(local_rank)
    sampler.start()
    timed(step, args.warmup)
    t0 = time.perf_counter()
    step_us = timed(step, K)
    t1 = time.perf_counter()
    calls = {"se_observe_decode": timed(observe, 30), "se_token_select": timed(select, 50),
             "se_token_decode": timed(lambda: reuse(0), 50)}
    e2e_us = timed(step_e2e, 30)
    sampler.stop()
    for ws in (obs.workspace, ws_tok):
        if binding.se_last_device_status(ws):
            raise SystemExit("device status %d" % binding.se_last_device_status(ws))
    n_tok = int(tok_cnt.sum().item())
    row = 2 * w0.D * 2
    qo = B * w0.H_q * (2 * w0.D + 4 * w0.D + 4)
    tok_bytes = n_tok * w0.H_kv * row + n_tok * 4 + qo
    obs_bytes = int(obs.sel_cnt.sum().item()) * 16 * row + qo + B * 16 * w0.max_pages * 4
    peak, peak_kind = measured_peak()
    gbs = tok_bytes / (calls["se_token_decode"] * 1e-6) / 1e9
    cb = None if args.no_cpu_baseline else omnikv_oracle_time(layers, budget, recent)
    splits = binding.se_decode_num_splits(p_tok)
    print(json.dumps({
        "metric": "omnikv_reuse_us_per_step", "value": step_us, "unit": "us", "n_gpus": 1, "steps": K,
        "warmup": args.warmup, "ms_per_step": step_us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w0.name, "B": B, "H_q": w0.H_q, "H_kv": w0.H_kv, "D": w0.D, "context_tokens": 32768,
                   "selected_tokens": budget, "recent_tokens": recent, "observation_layers": 1,
                   "sparse_layers": n_sparse, "storage_dtype": "bf16",
                   "l2": "inputs larger than L2 (%d MB read by the observation layer, %d MB per sparse layer)"
                         % (obs_bytes // 10**6, tok_bytes // 10**6)},
        "calls_us": calls,
        "algorithmic_bytes": {"se_observe_decode": obs_bytes, "se_token_decode": tok_bytes},
        "calls_gbs": {"se_observe_decode": obs_bytes / calls["se_observe_decode"] / 1e3,
                      "se_token_decode": gbs},
        "roofline": {"bound": "hbm", "kernel": "token_decode_kernel (se_token_decode)", "achieved": gbs, "peak": peak,
                     "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": gbs / peak,
                     "traffic": OMNIKV_NCU_TRAFFIC_BYTES if B == 24 else None, "algorithmic_bytes": tok_bytes},
        "clocks": sampler.summary(t0, t1),
        "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": sum(x.numel() * 2 for x in q_pin),
                "d2h_bytes_per_step": sum(x.numel() * 4 for x in o_pin)},
        "gpu_launches": K * (2 + 1 + n_sparse * (1 + int(splits > 1))) + K * int(binding.se_decode_num_splits(obs.p) > 1),
        "cpu_baseline": cb}))


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on the host cores, on the whole batch of the config
    (one layer; a multi-layer config is that time x layers).  Without a GPU to generate the pool on, a
    reduced batch is generated on the CPU and scaled by the page count (said in the sample string)."""
    import oracle
    n_layers = args.layers or (28 if args.config == 5 else 1)
    scale, note = 1.0, "whole batch, generated on the GPU and copied to the host"
    if torch.cuda.is_available():
        w = wl.CONFIGS[args.config]("cuda")
        w_cpu = w.to("cpu")
        del w
        torch.cuda.empty_cache()
    elif args.config in (3, 4, 5):
        kw = {3: dict(B=4), 4: dict(B=1, length=32768), 5: dict(B=8)}[args.config]
        w_cpu = wl.CONFIGS[args.config]("cpu", **kw)
        scale, note = 16.0, "no GPU: reduced batch generated on the CPU (%s), x16 to the full workload" % (kw,)
    else:
        w_cpu = wl.CONFIGS[args.config]("cpu")
        note = "whole batch, generated on the CPU"
    q, k, v = wl.bf16_bits(w_cpu.q), wl.bf16_bits(w_cpu.k_cache), wl.bf16_bits(w_cpu.v_cache)
    pt, sl = w_cpu.page_table.numpy(), w_cpu.seq_lens.numpy()
    meta = oracle.quest_meta(k, pt, sl, first_tok=np.zeros(w_cpu.B, np.int32))     # set-up: summaries after prefill
    u = None if w_cpu.score_accum is None else w_cpu.score_accum.numpy().astype(np.float64)
    steps = max(1, min(args.steps, 20))
    warm = max(1, min(args.warmup, 3))
    for _ in range(warm):
        oracle.decode_step(q, k, v, pt, sl, w_cpu.budget, meta=meta, u_accum=None if u is None else u.copy())
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.decode_step(q, k, v, pt, sl, w_cpu.budget, meta=meta, u_accum=None if u is None else u.copy())
    per = (time.perf_counter() - t0) / steps
    val = per * scale * n_layers * 1e6
    sample = "%d requests per step (%s), %.1f ms per oracle step%s" % (
        w_cpu.B, note, per * 1e3, "; one layer timed, x%d layers" % n_layers if n_layers > 1 else "")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "us", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": val / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w_cpu.name, "config_id": args.config, "layers": n_layers, "B": w_cpu.B,
                   "H_q": w_cpu.H_q, "H_kv": w_cpu.H_kv, "D": w_cpu.D, "page_size": 16,
                   "budget_tokens": w_cpu.budget, "storage_dtype": "bf16"},
        "cpu_baseline": {"value": val, "unit": "us", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


if __name__ == "__main__":
    main()
