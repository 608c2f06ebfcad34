"""The path shards by kv-head without any data-path collective: two gloo ranks on the CPU each run
their shard (here through the oracle; on GPUs each rank runs the CUDA path on its own device) and
the gathered shards must equal the unsharded result bit for bit."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_39068_b200 import workloads as wl
from helpers import host_arrays


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _make():
    return wl.build("tp", 970, 0, [300, 1000, 77], 8, 4, 32, 128, "cpu", permute_pool=True,
                    prune_fraction=0.1, with_score_accum=True)


def _run_shard(w):
    a = host_arrays(w)
    meta = oracle.quest_meta(a["k"], a["page_table"], a["seq_lens"], first_tok=np.zeros(w.B, np.int32))
    u = w.score_accum.numpy().astype(np.float64)
    res = oracle.decode_step(a["q"], a["k"], a["v"], a["page_table"], a["seq_lens"], w.budget, meta=meta, u_accum=u)
    return res["sel_idx"], res["out"], res["lse"], u


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        torch.set_num_threads(1)
        w = wl.shard_kv_heads(_make(), rank, world)
        sel, out, lse, u = _run_shard(w)
        gathered = [None] * world
        dist.all_gather_object(gathered, (sel, out, lse, u))       # test plumbing only, not the data path
        dist.barrier()
        if rank == 0:
            q.put(gathered)
    finally:
        dist.destroy_process_group()


def test_kv_head_shards_reproduce_the_unsharded_result():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    gathered = q.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sel_full, out_full, lse_full, u_full = _run_shard(_make())
    sel = np.concatenate([g[0] for g in gathered], axis=1)
    out = np.concatenate([g[1] for g in gathered], axis=1)
    lse = np.concatenate([g[2] for g in gathered], axis=1)
    u = np.concatenate([g[3] for g in gathered], axis=1)
    assert np.array_equal(sel, sel_full)
    assert np.array_equal(out, out_full) and np.array_equal(lse, lse_full)
    assert np.array_equal(u, u_full)
