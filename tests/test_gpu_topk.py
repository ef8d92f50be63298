"""GPU parity of specdec_verify_correct_topk (top-k sampling of Appendix D.1) against the CPU oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2405_19715_b200 import specdec, workloads as wl  # noqa: E402
from tests import parity  # noqa: E402


def _run(ctx, inp, k):
    t, d = specdec.from_numpy(inp["target_logits"]), specdec.from_numpy(inp["draft_logits"])
    B, K1, V = t.shape
    K = K1 - 1
    ratio = torch.full((B, K), -5.0, device="cuda")
    mass = torch.full((B,), -5.0, device="cuda")
    lens = None if inp.get("cand_len") is None else specdec.from_numpy(np.ascontiguousarray(inp["cand_len"], np.int32))
    n, tok = specdec.specdec_verify_correct_topk(
        ctx, t, d, specdec.from_numpy(np.ascontiguousarray(inp["cand_tokens"], np.int32)), lens,
        specdec.from_numpy(np.ascontiguousarray(inp["uniforms"], np.float32)), float(inp["temperature"]), k,
        accept_ratio=ratio, resid_mass=mass)
    torch.cuda.synchronize()
    return dict(n_accepted=n.cpu().numpy(), next_token=tok.cpu().numpy(), accept_ratio=ratio.cpu().numpy(),
                resid_mass=mass.cpu().numpy())


def _topk_tokens(inp, cfg, k):
    """Drafted tokens the way a top-k sampler would produce them: y ~ softmax of the draft's kept logits
    (Gumbel-max over the kept set), so that y lies in the draft's top-k."""
    rng = np.random.default_rng(cfg.seed + 999)
    d = inp["draft_logits"]
    df = (d.astype(np.uint32) << 16).view(np.float32) if d.dtype == np.uint16 else d
    df = np.nan_to_num(df.astype(np.float64), nan=-np.inf)
    kth = np.sort(df, axis=-1)[..., -min(k, df.shape[-1])][..., None]
    z = np.where(df >= kth, df / float(inp["temperature"]), -np.inf) + rng.gumbel(size=df.shape)
    return z.argmax(-1).astype(np.int32)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,k", [(7, 3), (33, 50), (1000, 50), (3000, 50), (4104, 1), (20000, 50), (32000, 256), (200000, 50), (262144, 7)])
def test_topk_small_shapes(V, k, dtype):
    B, K = 6, 5
    ctx = specdec.Context(B, K)
    cfg = wl.Workload("tk", B=B, K=K, V=V, dtype=dtype, sigma_d=2.5, sigma_n=1.0, T=0.9, ragged=True, seed=500 + V + k)
    inp = wl.make_verify_inputs(cfg, threads=1)
    y = _topk_tokens(inp, cfg, k)
    inp["cand_tokens"] = np.where(inp["cand_tokens"] >= 0, y, inp["cand_tokens"]).astype(np.int32)
    gpu = _run(ctx, inp, k)
    rep = parity.classify_rows(inp, gpu, dtype="f32", check_probs=False, top_k=k)
    assert rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == B and ctx.device_status() == 0
    ctx.close()


def test_topk_config_shapes_and_ties():
    """cfg3 (ragged, V=32000, bf16: many exact ties at the k-th value) and a slice of cfg4's shape with k=50;
    drafted tokens outside the target's kept set are rejected with certainty."""
    for name, B in (("cfg3", 64), ("cfg4", 24)):
        cfg = wl.CONFIGS[name].scaled(B=B)
        ctx = specdec.Context(cfg.B, cfg.K)
        inp = wl.make_verify_inputs(cfg)
        y = _topk_tokens(inp, cfg, 50)
        inp["cand_tokens"] = np.where(inp["cand_tokens"] >= 0, y, inp["cand_tokens"]).astype(np.int32)
        gpu = _run(ctx, inp, 50)
        rep = parity.classify_rows(inp, gpu, dtype="f32", check_probs=False, top_k=50)
        print(name, rep, "mean n", gpu["n_accepted"].mean())
        assert ctx.device_status() == 0
        gpu2 = _run(ctx, inp, 50)
        assert all(np.array_equal(gpu[k], gpu2[k]) for k in gpu)
        ctx.close()


def test_topk_adversarial_order_uses_the_exact_select():
    """Logits increasing along the vocabulary defeat the first-chunk bound (every later logit is a candidate):
    the kernel must fall back to its exact radix select and still agree with the oracle."""
    B, K, V = 3, 2, 50000
    ctx = specdec.Context(B, K)
    rng = np.random.default_rng(4)
    base = np.sort(rng.normal(scale=3, size=(B, K + 1, V)), axis=-1).astype(np.float32)
    d = (base[:, :K] + rng.normal(scale=0.01, size=(B, K, V))).astype(np.float32)
    inp = dict(target_logits=base, draft_logits=d, cand_tokens=np.full((B, K), V - 1, np.int32), cand_len=None,
               uniforms=wl.uniforms_24bit(rng, (B, K + 1)), temperature=np.float32(1.0))
    gpu = _run(ctx, inp, 50)
    parity.classify_rows(inp, gpu, dtype="f32", check_probs=False, top_k=50)
    assert ctx.device_status() == 0
    # k >= V is the unfiltered operation
    small = dict(inp, target_logits=base[:, :, :40].copy(), draft_logits=d[:, :, :40].copy(), cand_tokens=np.full((B, K), 39, np.int32))
    parity.classify_rows(small, _run(ctx, small, 64), dtype="f32", check_probs=False, top_k=None)
    # all logits equal: everything ties with the k-th largest -> flagged, not trapped
    flat = dict(inp, target_logits=np.zeros((B, K + 1, V), np.float32), draft_logits=np.zeros((B, K, V), np.float32))
    out = _run(ctx, flat, 50)
    assert ctx.device_status() == specdec.DATA_TOPK_TIES and np.all(out["n_accepted"] == -1)
    ctx.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_topk_with_a_masked_vocabulary(dtype):
    """Constrained decoding masks most logits with -inf: with fewer finite logits than k the filter keeps
    exactly the finite ones (the -inf entries carry no probability), and nothing is flagged."""
    B, K, V, k = 5, 3, 20000, 50
    ctx = specdec.Context(B, K)
    cfg = wl.Workload("mk", B=B, K=K, V=V, dtype=dtype, sigma_d=2.0, sigma_n=1.0, T=1.0, ragged=False, seed=321)
    inp = wl.make_verify_inputs(cfg, threads=1)
    rng = np.random.default_rng(9)
    allowed = np.sort(rng.choice(V, size=10, replace=False))
    neg = np.float32(-np.inf) if dtype == "f32" else np.uint16(0xFF80)
    for name in ("target_logits", "draft_logits"):
        a = inp[name]
        keep = a[..., allowed].copy()
        a[...] = neg
        a[..., allowed] = keep
    inp["cand_tokens"] = allowed[rng.integers(0, 10, size=(B, K))].astype(np.int32)
    gpu = _run(ctx, inp, k)
    rep = parity.classify_rows(inp, gpu, dtype="f32", check_probs=False, top_k=k)
    assert rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == B and ctx.device_status() == 0
    assert np.all(np.isin(gpu["next_token"], allowed))
    ctx.close()
