#!/usr/bin/env python
"""Benchmark of the sparse decode-attention hot path.

A *step* is one pass of the whole path over one batch of synthetic requests, per layer:
summary of the page holding each request's newest token -> page scores + top-k
(``se_page_select_fused`` does both; ``se_meta_update`` + ``se_page_select`` are the separate
calls) -> ``se_sparse_decode`` (split-K attention over the selected pages, LSE merge, optional
H2O statistic).  The default workload is the
continuous-batching mix (config 3: 64 requests, 4096..65536 tokens, 32/8 heads, D=128,
budget 2048, page tables permuted over one pool); ``--config`` picks another one.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

N > 1 is launched with torch.distributed.run, one rank per GPU; every rank runs the same
shape on its own data (the path shards by request / kv-head without any collective), so
scaling is weak.  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode kernel, from the ncu
# capture summarised in profiles/ (null until a capture of that workload exists)
NCU_TRAFFIC_BYTES = {
    # profiles/full_capture_config3_b24.md: 201.91 MB read for 24576 tiles, scaled to 65536 tiles,
    # plus the 1.06 MB of out/lse a full-size launch writes (it writes no partials: one split)
    "config3_contbatch_b64_mix": 539.5e6,
}
NCU_TRAFFIC_BYTES_SCORE = {
    # same capture: 244.97 MB read + 5.07 MB written for 249.3 MB of summaries, scaled to 561.5 MB
    "config3_contbatch_b64_mix": 563.2e6,
}


# dram bytes of one h2o_compact_kernel launch on the 64-request eviction workload (profiles/)
H2O_NCU_TRAFFIC_BYTES = 2055e6        # 770.7 MB at 24 requests, scaled by the request count


# dram bytes of one token_decode_kernel launch on the 24-request selection-reuse workload (profiles/)
OMNIKV_NCU_TRAFFIC_BYTES = 209e6     # 69.8 MB at 8 requests, scaled by the request count


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


def make_layers(config: int, device, n_layers: int, rank: int, batch: int = 0):
    fn = wl.CONFIGS[config]
    if batch:
        base = fn
        fn = lambda device, layer=0: base(device, layer=layer, B=batch)
    layers = []
    first = None
    for l in range(n_layers):
        w = fn(device, layer=l + 100 * rank) if config != 5 else fn(device, layer=l)
        if first is None:
            first = w
        else:                                 # the block table is per request, shared by all layers
            w.page_table, w.seq_lens = first.page_table, first.seq_lens
        layers.append(w)
    return layers


# ------------------------------------------------------------------ CPU oracle timing
def oracle_time(w, target_s=(10.0, 30.0)):
    """Times the oracle, as it stands, on a bounded sample of the workload's requests and
    scales to the full batch by the number of (present + selected) pages."""
    import oracle
    order = list(range(0, w.B, max(1, w.B // 16)))[:16]
    sub = wl.sub_workload(w, order, "cpu")
    q, k, v = wl.bf16_bits(sub.q), wl.bf16_bits(sub.k_cache), wl.bf16_bits(sub.v_cache)
    pt, sl = sub.page_table.numpy(), sub.seq_lens.numpy()
    meta = oracle.quest_meta(k, pt, sl, first_tok=np.zeros(sub.B, np.int32))
    u = None if sub.score_accum is None else sub.score_accum.numpy().astype(np.float64)
    times = []
    t_begin = time.perf_counter()
    while len(times) < 3 or time.perf_counter() - t_begin < target_s[0]:
        t0 = time.perf_counter()
        oracle.decode_step(q, k, v, pt, sl, sub.budget, meta=meta, u_accum=u)
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_begin > target_s[1]:
            break
    n_all = (w.seq_lens.cpu().numpy() + 15) // 16
    n_sub = (sl + 15) // 16
    scale = float(n_all.sum()) / float(n_sub.sum())
    best = min(times)
    return dict(value=best * scale * 1e6, unit="us", cores=oracle.num_threads(), kind="oracle",
                sample="%d of %d requests (every %d-th), fp64 C oracle with OpenMP over (request, kv-head), "
                       "best of %d runs (%.0f s of wall time) = %.1f ms, scaled x%.2f by page count to the full batch"
                       % (sub.B, w.B, max(1, w.B // 16), len(times), time.perf_counter() - t_begin, best * 1e3, scale),
                sample_seconds=best)


# ------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=3, choices=sorted(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="layers per step (default 1; 28 for config 5)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=0,
                    help="override the number of requests (configs 3-5; for small profiling captures)")
    ap.add_argument("--no-graph", action="store_true", help="launch the calls directly instead of a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="decode", choices=["decode", "h2o_evict", "omnikv_reuse"],
                    help="decode = the sparse decode step (the headline); h2o_evict = one H2O eviction "
                         "(retained set + in-place compaction) of 64 requests, 5120 -> 4096 tokens; "
                         "omnikv_reuse = one observation layer (full attention + token selection) and four "
                         "sparse layers reusing its 2048+32 tokens, 24 requests of 32768 tokens")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    n_layers = args.layers or (28 if args.config == 5 else 1)

    if args.workload in ("h2o_evict", "omnikv_reuse"):
        if rank == 0:                        # these steps have no multi-GPU leg of their own
            (run_h2o_evict if args.workload == "h2o_evict" else run_omnikv)(args, local_rank)
        return
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, n_layers)
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

    layers = make_layers(args.config, dev, n_layers, rank, args.batch)
    h2o = layers[0].score_accum is not None
    states = [binding.DecodeState(w) for w in layers]
    accums = [w.score_accum.clone() if h2o else None for w in layers]
    for st in states:
        st.rebuild_meta()
    torch.cuda.synchronize()

    def step():
        for st, u in zip(states, accums):
            st.step(score_accum=u)

    step()
    torch.cuda.synchronize()
    for st in states:
        if st.status() != 0:
            raise SystemExit("device status word not clean")
    bytes_l = [algorithmic_bytes(st.w, st.sel_cnt, h2o) for st in states]
    total_bytes = sum(b["total"] for b in bytes_l)
    working_set = total_bytes
    flush = working_set < 2 * L2_BYTES
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if flush else None
    flush_src = torch.zeros(2 * L2_BYTES // 4, dtype=torch.int32, device=dev) if flush else None
    flush_sink = torch.zeros(1, dtype=torch.int32, device=dev) if flush else None

    def flush_l2(i):
        """Evicts the step's data from L2: a 252 MiB write, then a 252 MiB read of another buffer, so that
        the lines the timed step displaces are clean (displacing the write's dirty lines would charge
        the step one write-back per byte it reads)."""
        flush_buf.fill_(i & 0xFF)
        flush_sink.copy_(flush_src.max().reshape(1))

    graph = None
    if not args.no_graph:
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            step()
        torch.cuda.current_stream().wait_stream(s)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
    run_step = graph.replay if graph is not None else step

    sampler = ClockSampler(local_rank)
    sampler.start()

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        run_step()
    barrier()
    K = args.steps
    t_wall0 = time.perf_counter()
    if flush:
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        ends = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        for i in range(K):
            flush_l2(i)
            starts[i].record()
            run_step()
            ends[i].record()
        barrier()
        total_ms = sum(a.elapsed_time(b) for a, b in zip(starts, ends))
    else:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(K):
            run_step()
        e1.record()
        barrier()
        total_ms = e0.elapsed_time(e1)
    t_wall1 = time.perf_counter()
    if world > 1:
        t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / K
    clocks = sampler.summary(t_wall0, t_wall1)

    # ---- per-call timing (same stream, CUDA events, each call in its own loop)
    def time_call(fn, iters):
        for _ in range(3):
            fn()
        if flush:
            tot = 0.0
            for i in range(iters):
                flush_l2(i)
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
    st0, u0 = states[0], accums[0]
    call_us = {
        "se_meta_update": time_call(st0.update_meta, iters),
        "se_page_select": time_call(st0.select, iters),
        "se_page_select_scores": time_call(lambda: st0.select(entry="se_page_select_scores"), iters),
        "se_page_select_topk": time_call(lambda: st0.select(entry="se_page_select_topk"), iters),
        "se_page_select_fused": time_call(st0.select_fused, iters),
        "se_decode_step": time_call(lambda: st0.step(u0), iters),
        "se_sparse_decode": time_call(lambda: st0.decode(u0), iters),
        "se_sparse_decode_splits": time_call(lambda: st0.decode(u0, entry="se_sparse_decode_splits"), iters),
        "se_combine": time_call(lambda: st0.decode(u0, entry="se_combine"), iters),
    }
    b0 = bytes_l[0]
    peak, peak_kind = measured_peak()
    # the dominant kernel, timed on its own: decode_kernel is all that se_sparse_decode_splits launches
    dec_gbs = b0["decode_kernel"] / (call_us["se_sparse_decode_splits"] * 1e-6) / 1e9
    sel_gbs = b0["select_call"] / (call_us["se_page_select"] * 1e-6) / 1e9
    score_gbs = b0["select_call"] / (call_us["se_page_select_scores"] * 1e-6) / 1e9
    rl_decode = {"bound": "hbm", "kernel": "decode_kernel (se_sparse_decode_splits)", "achieved": dec_gbs,
                 "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": dec_gbs / peak,
                 "traffic": NCU_TRAFFIC_BYTES.get(layers[0].name), "algorithmic_bytes": b0["decode_kernel"],
                 "us": call_us["se_sparse_decode_splits"]}
    rl_score = {"bound": "hbm", "kernel": "score_kernel (se_page_select_scores)", "achieved": score_gbs,
                "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s", "frac": score_gbs / peak,
                "traffic": NCU_TRAFFIC_BYTES_SCORE.get(layers[0].name), "algorithmic_bytes": b0["select_call"],
                "us": call_us["se_page_select_scores"]}
    # the dominant kernel is whichever of the two streaming kernels takes longer on this workload
    rl_main, rl_other = (rl_score, rl_decode) if rl_score["us"] >= rl_decode["us"] else (rl_decode, rl_score)
    step_gbs = total_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end through the public API with host buffers: the step's inputs (q, lengths, page
    # table) sit in one pinned block and go up in one copy, out + lse come back in one copy
    import copy

    def packed(tensors, device, pin):
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

    e2e_states, host_in, dev_in, host_out, dev_out = [], [], [], [], []
    for w, st in zip(layers, states):
        ins = [w.q, w.seq_lens, w.page_table]
        hb, hv = packed(ins, "cpu", True)
        db, dv = packed(ins, dev, False)
        for src, h, d in zip(ins, hv, dv):
            h.copy_(src)
            d.copy_(src)
        outs = [st.out, st.lse]
        ob, ov = packed(outs, dev, False)
        hob, _ = packed(outs, "cpu", True)
        st2 = copy.copy(st)                       # same params, workspace, summaries and selection buffers
        st2.w = dataclasses.replace(w, q=dv[0], seq_lens=dv[1], page_table=dv[2])
        st2.out, st2.lse = ov
        e2e_states.append(st2)
        host_in.append(hb); dev_in.append(db); host_out.append(hob); dev_out.append(ob)
    h2d = sum(b.numel() for b in host_in)
    d2h = sum(b.numel() for b in host_out)

    def e2e_body():
        for st2, u, hb, db, ob, hob in zip(e2e_states, accums, host_in, dev_in, dev_out, host_out):
            db.copy_(hb, non_blocking=True)
            st2.step(score_accum=u)
            hob.copy_(ob, non_blocking=True)

    # the way a serving loop drives the library: the host fills fixed pinned buffers, one graph launch
    # does upload + step + download, and the host waits for the result before the next step
    e2e_graph = None
    if not args.no_graph:
        s2 = torch.cuda.Stream()
        s2.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s2):
            e2e_body()
        torch.cuda.current_stream().wait_stream(s2)
        torch.cuda.synchronize()
        e2e_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(e2e_graph):
            e2e_body()

    def e2e_step():
        if e2e_graph is not None:
            e2e_graph.replay()
        else:
            e2e_body()
        torch.cuda.synchronize()

    for _ in range(3):
        e2e_step()
    e2e_iters = max(10, min(K, 200))
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(e2e_iters):
        if flush:
            flush_l2(i)
        e2e_step()
    b.record()
    barrier()
    e2e_ms = a.elapsed_time(b) / e2e_iters
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        e2e_ms = float(t.item())
    sampler.stop()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_time(layers[0])
        if n_layers > 1:
            cpu_baseline["value"] *= n_layers
            cpu_baseline["sample"] += "; one layer timed, x%d layers" % n_layers

    if rank == 0:
        # score, top-k, decode (summary update fused into score); the merge kernel runs only when
        # the pairs are split or the H2O epilogue is on
        launches_per_step = n_layers * binding.se_decode_step_launches(states[0].p, layers[0].budget, h2o)
        line = {
            "metric": METRIC, "value": ms_per_step * 1e3, "unit": "us", "n_gpus": world,
            "steps": K, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": layers[0].name, "config_id": args.config, "layers": n_layers,
                "B": layers[0].B, "H_q": layers[0].H_q, "H_kv": layers[0].H_kv, "D": layers[0].D,
                "page_size": 16, "budget_tokens": layers[0].budget, "storage_dtype": "bf16",
                "present_pages": b0["present_pages"], "selected_pages": b0["selected_pages"],
                "h2o_epilogue": h2o, "cuda_graph": graph is not None,
                "l2": ("flushed before every step: a %d MiB write, then a %d MiB read (leaves clean lines)" % (2 * L2_BYTES >> 20, 2 * L2_BYTES >> 20)) if flush
                      else "inputs larger than L2 (%.0f MB touched per step)" % (working_set / 1e6),
                "parallelism": "1 GPU" if world == 1 else "%d replicas, no collective" % world,
                "global_batch": layers[0].B * world,
                "checksums_layer0": checksums(layers[0]),
            },
            "algorithmic_bytes_per_step": total_bytes,
            "achieved_gbs": step_gbs * world,
            "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
            "frac_of_measured_copy": step_gbs / peak,
            "calls_us": call_us,
            "calls_gbs": {"se_page_select": sel_gbs, "se_sparse_decode": dec_gbs},
            "roofline": rl_main,
            "roofline_second_kernel": rl_other,
            "clocks": clocks,
            "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * K,
            "cpu_baseline": cpu_baseline,
        }
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


def run_reference(args, n_layers):
    """Reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload."""
    import oracle
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    if dev == "cpu" and args.config in (3, 4, 5):
        kw = {3: dict(B=4), 4: dict(B=1, length=32768), 5: dict(B=8)}[args.config]
        w = wl.CONFIGS[args.config](dev, **kw)
        # no GPU to generate the full pool on: a sixteenth of the workload, scaled back up
        reduced = 16.0
        note = "generated on the CPU at reduced size (%s), then x%.0f to the full workload" % (kw, reduced)
    else:
        w = wl.CONFIGS[args.config](dev)
        reduced = 1.0
        note = "full workload generated on the GPU, sample copied to the host"
    order = list(range(0, w.B, max(1, w.B // 16)))[:16]
    sub = wl.sub_workload(w, order, "cpu")
    q, k, v = wl.bf16_bits(sub.q), wl.bf16_bits(sub.k_cache), wl.bf16_bits(sub.v_cache)
    pt, sl = sub.page_table.numpy(), sub.seq_lens.numpy()
    meta = oracle.quest_meta(k, pt, sl, first_tok=np.zeros(sub.B, np.int32))
    u = None if sub.score_accum is None else sub.score_accum.numpy().astype(np.float64)
    n_all = (w.seq_lens.cpu().numpy() + 15) // 16
    scale = float(n_all.sum()) / float(((sl + 15) // 16).sum()) * n_layers * reduced
    steps = max(1, min(args.steps, 20))
    warm = max(1, min(args.warmup, 3))
    for _ in range(warm):
        oracle.decode_step(q, k, v, pt, sl, sub.budget, meta=meta, u_accum=u)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.decode_step(q, k, v, pt, sl, sub.budget, meta=meta, u_accum=u)
    per = (time.perf_counter() - t0) / steps
    val = per * scale * 1e6
    sample = ("%d of %d requests per step (%s), %.1f ms per sample step, scaled x%.2f by page count%s"
              % (sub.B, w.B, note, per * 1e3, scale, " and layers" if n_layers > 1 else ""))
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "us", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": val / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "config_id": args.config, "layers": n_layers},
        "cpu_baseline": {"value": val, "unit": "us", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


if __name__ == "__main__":
    main()
