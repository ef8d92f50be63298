"""GPU parity of vocabulary-sharded verify/correct against the oracle on the concatenated logits.
The ranks are emulated on one GPU by running each phase for every shard in turn (no kernel of this
path waits for another launch), with the all-gathers done as stacks."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2405_19715_b200 import sharded, specdec, workloads as wl  # noqa: E402
from tests import parity  # noqa: E402


def run_sharded(ctx, inp, slices):
    """The protocol of paper_2405_19715_b200.sharded with world = len(slices), on one GPU."""
    V = inp["target_logits"].shape[2]
    T = float(inp["temperature"])
    B, K = inp["cand_tokens"].shape
    tok = specdec.from_numpy(np.ascontiguousarray(inp["cand_tokens"], np.int32))
    lens = None if inp.get("cand_len") is None else specdec.from_numpy(np.ascontiguousarray(inp["cand_len"], np.int32))
    uni = specdec.from_numpy(np.ascontiguousarray(inp["uniforms"], np.float32))
    shards = [(specdec.from_numpy(np.ascontiguousarray(inp["target_logits"][:, :, o:o + s])),
               specdec.from_numpy(np.ascontiguousarray(inp["draft_logits"][:, :, o:o + s])), o) for o, s in slices]
    stats_all = torch.stack([specdec.specdec_shard_stats(ctx, t, d, o, V, tok, lens, T) for t, d, o in shards])
    ratio = torch.full((B, K), -5.0, device="cuda")
    acc = [specdec.specdec_shard_accept(ctx, t, d, o, V, stats_all, lens, uni, T, accept_ratio=ratio) for t, d, o in shards]
    for n, norm, _ in acc[1:]:                                  # replicated results agree bit for bit
        assert torch.equal(n, acc[0][0]) and torch.equal(norm, acc[0][1])
    mass_all = torch.stack([m for _, _, m in acc])
    rm = torch.full((B,), -5.0, device="cuda")
    toks = torch.stack([specdec.specdec_shard_draw(ctx, t, d, o, V, stats_all, mass_all, r, acc[r][0], lens, uni,
                                                   acc[r][1], T, resid_mass=rm)
                        for r, (t, d, o) in enumerate(shards)])
    torch.cuda.synchronize()
    owners = (toks >= 0).sum(0)
    return dict(n_accepted=acc[0][0].cpu().numpy(), next_token=toks.max(0).values.cpu().numpy(),
                accept_ratio=ratio.cpu().numpy(), resid_mass=rm.cpu().numpy()), owners.cpu().numpy()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,cuts", [(1000, [1000]), (1000, [333, 667]), (1003, [400, 800]), (32000, [8000, 16000, 24000]),
                                    (4096, [8, 16, 4088])])
def test_sharded_matches_oracle(V, cuts, dtype):
    B, K = 10, 6
    ctx = specdec.Context(B, K)
    cfg = wl.Workload("sh", B=B, K=K, V=V, dtype=dtype, sigma_d=2.0, sigma_n=1.0, T=0.9, ragged=True, seed=70 + V + len(cuts))
    inp = wl.make_verify_inputs(cfg, threads=1)
    edges = [0] + [c for c in cuts if c < V] + [V]
    slices = [(a, b - a) for a, b in zip(edges[:-1], edges[1:])]
    gpu, owners = run_sharded(ctx, inp, slices)
    assert np.all(owners == 1)                                   # exactly one rank draws each row
    rep = parity.classify_rows(inp, gpu, dtype=dtype, check_probs=False)
    assert rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == B and ctx.device_status() == 0
    ctx.close()


def test_sharded_config_shapes():
    """cfg3 (ragged, 64 rows) over 4 ranks and a slice of cfg4 (V = 128256) over 8 ranks."""
    for name, B, world in (("cfg3", 64, 4), ("cfg4", 16, 8)):
        cfg = wl.CONFIGS[name].scaled(B=B)
        ctx = specdec.Context(cfg.B, cfg.K)
        inp = wl.make_verify_inputs(cfg)
        gpu, owners = run_sharded(ctx, inp, sharded.vocab_slices(cfg.V, world))
        assert np.all(owners == 1)
        rep = parity.classify_rows(inp, gpu, dtype=cfg.dtype, check_probs=False)
        print(name, rep)
        assert ctx.device_status() == 0
        ctx.close()


def test_sharded_special_cases():
    B, K, V = 6, 4, 512
    ctx = specdec.Context(B, K)
    rng = np.random.default_rng(5)
    t = rng.normal(scale=2, size=(B, K + 1, V)).astype(np.float32)
    base = dict(target_logits=t, draft_logits=t[:, :K].copy(), cand_tokens=rng.integers(0, V, (B, K)).astype(np.int32),
                cand_len=None, uniforms=wl.uniforms_24bit(rng, (B, K + 1)), temperature=np.float32(1.0))
    slices = [(0, 128), (128, 256), (384, 128)]
    gpu, owners = run_sharded(ctx, base, slices)                 # p == q: everything accepted, bonus draw
    assert np.all(gpu["n_accepted"] == K) and np.all(owners == 1)
    parity.classify_rows(base, gpu, dtype="f32", check_probs=False)
    # a drafted token outside the vocabulary marks its row bad and nothing else
    bad = dict(base, cand_tokens=base["cand_tokens"].copy())
    bad["cand_tokens"][2, 1] = V + 3
    gpu, _ = run_sharded(ctx, bad, slices)
    assert gpu["n_accepted"][2] == -1 and gpu["next_token"][2] == -1 and ctx.device_status() == specdec.DATA_BAD_TOKEN
    assert np.all(np.delete(gpu["n_accepted"], 2) == K)
    ctx.close()


def test_sharded_argument_errors():
    ctx = specdec.Context(4, 2)
    t = torch.zeros(4, 3, 64, device="cuda")
    d = torch.zeros(4, 2, 64, device="cuda")
    tok = torch.zeros(4, 2, dtype=torch.int32, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:               # columns beyond the vocabulary
        specdec.specdec_shard_stats(ctx, t, d, 32, 64, tok, None, 1.0)
    assert e.value.code == specdec.EINVAL
    ctx.close()
