"""The multi-GPU leg of the benchmark shards batch rows across ranks with no data-path collective;
only the timing maximum and the token count cross ranks.  Checked here with two gloo ranks on CPU."""
import os
import sys
from pathlib import Path

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from oracle import specdec_oracle as orc
    from paper_2405_19715_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.shard_config(wl.Workload("dist", B=3, K=4, V=64, dtype="bf16", sigma_d=2.0, sigma_n=1.0, T=1.0,
                                         ragged=True, seed=7), rank)
    inp = wl.make_verify_inputs(cfg, threads=1)
    o = orc.verify_correct(inp["target_logits"], inp["draft_logits"], inp["cand_tokens"], inp["cand_len"],
                           inp["uniforms"], inp["temperature"])
    ms, tokens = bench.aggregate(10.0 + rank, float(inp["cand_len"].sum()), world, torch.device("cpu"))
    bench.barrier(world)
    out.put((rank, ms, tokens, int(inp["cand_len"].sum()), inp["target_logits"][:, 0, :4].tolist(), o["n_accepted"].tolist()))
    dist.destroy_process_group()


def test_two_rank_sharding_and_aggregation():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, tok0, own0, head0, n0), (r1, ms1, tok1, own1, head1, n1) = res
    assert ms0 == ms1 == 11.0                      # the slowest rank's time
    assert tok0 == tok1 == own0 + own1             # tokens of the whole job
    assert head0 != head1                          # each rank drew its own rows
    assert len(n0) == len(n1) == 3


def test_launcher_starts_the_ranks_itself():
    """`python bench.py --gpus 2` without a launcher around it: the script starts two ranks on 127.0.0.1,
    each learns its rank and the world size, and rank 0 prints one line for the whole job."""
    import json
    import bench
    rc, out = bench.launch_ranks(2, ["--gpus", "2", "--stub-step", "--steps", "3"], extra_env={"NCCL_DEBUG": "WARN"})
    assert rc == 0, out
    lines = [ln for ln in out.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["stub"] is True
    assert sorted(map(tuple, line["ranks_seen"])) == [(0, 2), (1, 2)]
    assert line["tokens_per_step"] == 30.0                        # 10 + 20: summed over the ranks
