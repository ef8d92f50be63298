"""GPU parity of specdec_verify_greedy (Section 4.1's greedy setting) against the CPU oracle: integer
outputs, compared exactly."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import specdec_oracle as orc  # noqa: E402
from paper_2405_19715_b200 import specdec, workloads as wl  # noqa: E402


def _run(ctx, target, y, lens):
    t = specdec.from_numpy(target)
    B, K1, _ = t.shape
    am = torch.full((B, K1), -9, dtype=torch.int32, device="cuda")
    n, tok = specdec.specdec_verify_greedy(ctx, t, specdec.from_numpy(np.ascontiguousarray(y, np.int32)),
                                           None if lens is None else specdec.from_numpy(np.ascontiguousarray(lens, np.int32)),
                                           target_argmax=am)
    torch.cuda.synchronize()
    return n.cpu().numpy(), tok.cpu().numpy(), am.cpu().numpy()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 7, 33, 1000, 4104, 32000])
def test_greedy_matches_oracle(V, dtype):
    B, K = 9, 6
    ctx = specdec.Context(B, K)
    cfg = wl.Workload("g", B=B, K=K, V=V, dtype=dtype, sigma_d=2.0, sigma_n=0.6, T=1.0, ragged=True, seed=300 + V)
    inp = wl.make_verify_inputs(cfg, threads=1)
    target, lens = inp["target_logits"], inp["cand_len"]
    # greedy drafts: the draft's argmax where the draft row exists, anything elsewhere
    d64 = orc.logits_to_f64(inp["draft_logits"])
    y = np.where(np.isnan(d64).all(-1), 0, np.nan_to_num(d64, nan=-np.inf).argmax(-1)).astype(np.int32)
    n, tok, am = _run(ctx, target, y, lens)
    on, otok, oam = orc.greedy_verify_tokens(target, y, lens)
    assert np.array_equal(n, on) and np.array_equal(tok, otok) and np.array_equal(am, oam)
    assert ctx.device_status() == 0
    assert (on < lens).any() or V == 1
    ctx.close()


def test_greedy_ties_resolve_to_lowest_index_and_full_acceptance():
    B, K, V = 4, 5, 4096
    ctx = specdec.Context(B, K)
    rng = np.random.default_rng(0)
    t = np.round(rng.normal(size=(B, K + 1, V)) * 2).astype(np.float32)       # heavy ties
    y = t[:, :K].argmax(-1).astype(np.int32)                                   # numpy: first maximum
    n, tok, am = _run(ctx, t, y, None)
    assert np.all(n == K) and np.array_equal(tok, t[:, K].argmax(-1)) and np.array_equal(am, t.argmax(-1))
    y2 = y.copy()
    y2[:, 2] = (y2[:, 2] + 1) % V
    n, tok, _ = _run(ctx, t, y2, None)
    assert np.all(n == 2) and np.array_equal(tok, t[:, 2].argmax(-1))
    ctx.close()


def test_greedy_bad_data_and_large_shape():
    cfg = wl.CONFIGS["cfg3"]
    ctx = specdec.Context(cfg.B, cfg.K)
    inp = wl.make_verify_inputs(cfg)
    y = np.maximum(inp["cand_tokens"], 0)
    n, tok, am = _run(ctx, inp["target_logits"], y, inp["cand_len"])
    on, otok, oam = orc.greedy_verify_tokens(inp["target_logits"], y, inp["cand_len"])
    assert np.array_equal(n, on) and np.array_equal(tok, otok) and np.array_equal(am, oam)
    lens = inp["cand_len"].copy()
    lens[3] = cfg.K + 2
    y[5, 0] = cfg.V + 1
    n, tok, _ = _run(ctx, inp["target_logits"], y, lens)
    assert n[3] == -1 and tok[3] == -1 and n[5] == -1 and tok[5] == -1
    assert ctx.device_status() == (specdec.DATA_BAD_LENGTH | specdec.DATA_BAD_TOKEN)
    ctx.close()
