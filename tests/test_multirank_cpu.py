"""The N > 1 host path on CPU: two gloo ranks take disjoint requests, agree on the slowest rank's
time and exchange their budgets.  (The pass itself has no collective; see shard.py.)"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import gvote_oracle as o
from paper_2509_03136_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    base = synth.make_small(7, seq_lens=(48, 33), S=3)
    cfg = shard.rank_workload(base, rank)
    li = synth.make_layer(cfg, 0)
    res, _, _ = o.compress_layer(li.h, li.W_q, li.b_q, li.K, li.V, li.cu_seqlens, n_q_heads=cfg.n_q_heads,
                                 d_k=cfg.d_k, theta=cfg.rope_theta, S=cfg.S, p_nuc=cfg.p_nuc, n_f=cfg.n_f,
                                 n_s=cfg.n_s, seed=cfg.seed, layer_id=0)
    budget = torch.tensor(np.stack([r.budget for r in res]), dtype=torch.int32)
    slowest = shard.max_over_ranks(1.0 + rank, dist)
    gathered = shard.gather_budgets(budget, dist)
    torch.save({"seed": cfg.seed, "slowest": slowest, "own": budget, "all": gathered,
                "h0": float(li.h[0, 0])}, os.path.join(out_dir, f"r{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_disjoint_requests_max_time_and_budget_gather(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(tmp_path / f"r{i}.pt") for i in range(world)]
    assert r[0]["seed"] != r[1]["seed"] and r[0]["h0"] != r[1]["h0"]          # different requests
    assert r[0]["slowest"] == r[1]["slowest"] == 2.0                            # max over ranks
    for i in range(world):
        for j in range(world):
            assert torch.equal(r[i]["all"][j], r[j]["own"])                     # everyone sees everyone's budgets
    assert shard.job_throughput(1000, 2, 0.5) == 4000.0


def test_single_process_is_a_no_op():
    assert shard.max_over_ranks(3.5) == 3.5
    b = torch.ones(1, 2, dtype=torch.int32)
    assert shard.gather_budgets(b)[0] is b


def test_bench_starts_its_own_ranks_only_when_no_launcher_did():
    """`bench.py --gpus N` without a launcher's environment re-launches itself under torch.distributed.run
    with one process per GPU on 127.0.0.1; under a launcher, or for one GPU, it runs as it is."""
    argv = ["--gpus", "4", "--steps", "3"]
    cmd = shard.self_launch_command("/x/bench.py", argv, 4, {}, port=29511)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511" and cmd[-5:] == ["/x/bench.py"] + argv
    assert shard.self_launch_command("/x/bench.py", argv, 4, {"WORLD_SIZE": "4", "RANK": "1"}) is None
    assert shard.self_launch_command("/x/bench.py", ["--gpus", "1"], 1, {}) is None
    port = int(shard.self_launch_command("/x/bench.py", argv, 2, {})[8])       # a free port is picked when none is given
    assert 1024 < port < 65536
