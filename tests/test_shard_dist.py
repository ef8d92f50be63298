"""The exchange protocol of vocabulary-sharded verify/correct (two all-gathers and a max-reduction
around three local phases) on two and three gloo ranks, with a float64 CPU model of the phases in
place of the CUDA binding; the protocol's result must equal the oracle on the concatenated logits."""
import os
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _worker(rank, world, port, out):
    try:
        _run(rank, world, port, out)
    except Exception as e:                                      # report instead of leaving the parent to time out
        out.put((rank, "error", repr(e)))
        raise


def _run(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2405_19715_b200 import sharded, workloads as wl
    from tests import shard_model
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.Workload("vs", B=12, K=5, V=96, dtype="f32", sigma_d=2.0, sigma_n=1.2, T=0.9, ragged=True, seed=31)
    inp = wl.make_verify_inputs(cfg, threads=1)                 # replicated: every rank generates the same job
    off, size = sharded.vocab_slices(cfg.V, world, multiple=4)[rank]
    ts = torch.from_numpy(np.ascontiguousarray(inp["target_logits"][:, :, off:off + size]))
    ds = torch.from_numpy(np.ascontiguousarray(inp["draft_logits"][:, :, off:off + size]))
    n, tok = sharded.verify_correct_vocab_sharded(
        None, ts, ds, off, cfg.V, torch.from_numpy(inp["cand_tokens"]), torch.from_numpy(inp["cand_len"].astype(np.int32)),
        torch.from_numpy(inp["uniforms"]), float(inp["temperature"]), ops=shard_model)
    out.put((rank, n.tolist(), tok.tolist()))
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_vocab_sharded_protocol_matches_the_oracle(world):
    from oracle import specdec_oracle as orc
    from paper_2405_19715_b200 import workloads as wl
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() * 7 + world) % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = wl.Workload("vs", B=12, K=5, V=96, dtype="f32", sigma_d=2.0, sigma_n=1.2, T=0.9, ragged=True, seed=31)
    inp = wl.make_verify_inputs(cfg, threads=1)
    o = orc.verify_correct(inp["target_logits"], inp["draft_logits"], inp["cand_tokens"], inp["cand_len"],
                           inp["uniforms"], inp["temperature"])
    assert all(r[1] != "error" for r in res), res
    for rank, n, tok in res:                                    # every rank ends with the whole answer
        assert n == o["n_accepted"].tolist(), f"rank {rank}"
        assert tok == o["next_token"].tolist(), f"rank {rank}"
    assert len(set(o["n_accepted"].tolist())) > 1               # the job has rejections and full acceptances


def test_vocab_slices():
    from paper_2405_19715_b200 import sharded
    assert sharded.vocab_slices(128256, 8) == [(i * 16032, 16032) for i in range(8)]
    s = sharded.vocab_slices(32000, 3)
    assert sum(sz for _, sz in s) == 32000 and all(sz % 8 == 0 for _, sz in s[:-1]) and s[1][0] == s[0][1]
    with pytest.raises(ValueError):
        sharded.vocab_slices(16, 4, multiple=8)
