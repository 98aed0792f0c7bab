"""World-size-2 run of the multi-rank bookkeeping on CPU (gloo): each rank plans its own prompt through
the C ABI and the job totals are the sum of tokens and the maximum of times.  No data-path collective
exists in this pass, so this is the whole N > 1 host logic."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2507_06517_b200 import binding as B
    from paper_2507_06517_b200 import sharding, synth
    wl = sharding.rank_workload(synth.workload("C4"), rank)
    cfg = B.Config(wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window, wl.n_shallow,
                   reserve_ratio=wl.budget_frac)
    _, _, k = B.spindlekv_plan_layers(cfg, wl.seq_lens)
    k0, _ = synth.unit_kv(wl.replace(seq_lens=(64,)), 0, 0, 0)
    tokens, ms = sharding.aggregate(wl.total_tokens, 10.0 * (rank + 1), dist)
    out[rank] = (tokens, ms, int(k.sum()), float(k0[0, 0]), wl.total_tokens)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_aggregate_and_plan_independently():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == res[0][4] + res[1][4]   # tokens: sum over ranks
    assert res[0][1] == res[1][1] == 20.0                      # time: max over ranks
    assert res[0][2] == res[1][2]                              # same shape, same plan
    assert res[0][3] != res[1][3]                              # different prompts (seeds)


def test_single_process_aggregate_is_identity():
    from paper_2507_06517_b200 import sharding
    assert sharding.aggregate(123, 4.5) == (123, 4.5)
    assert sharding.throughput(1000, 2, 500.0) == 4000.0
