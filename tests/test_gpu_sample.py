"""GPU parity of specdec_sample (Algorithm 1's draw y ~ q; the K = 0 round of Algorithm 2) against the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import specdec_oracle as orc  # noqa: E402
from paper_2405_19715_b200 import specdec, workloads as wl  # noqa: E402
from tests import parity  # noqa: E402


def _case(B, V, dtype, seed, T=0.8):
    cfg = wl.Workload("s", B=B, K=1, V=V, dtype=dtype, sigma_d=2.0, sigma_n=1.0, T=T, ragged=False, seed=seed)
    inp = wl.make_verify_inputs(cfg, threads=1)
    logits = np.ascontiguousarray(inp["draft_logits"][:, 0])
    u = np.ascontiguousarray(inp["uniforms"][:, 0])
    return logits, u, T


def _check(logits, u, T, top_k, got):
    """Exact match, or a draw within 1e-6 of a CDF boundary of the token the GPU chose."""
    z = orc.logits_to_f64(logits)
    want = orc.sample(logits, u, T, top_k)
    boundary = 0
    for b in np.nonzero(want != got)[0]:
        w = orc.sampling_weights(z[b], None, T, top_k)
        F = np.cumsum(w) / w.sum()
        g = int(got[b])
        assert 0 <= g < len(w) and w[g] > 0, f"row {b}: token {g} has no weight"
        lo = F[g - 1] if g > 0 else 0.0
        assert lo - 1e-6 <= u[b] <= F[g] + 1e-6, f"row {b}: token {g} vs {want[b]}, u={u[b]}"
        boundary += 1
    return boundary


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,top_k", [(5, 0), (1000, 0), (4099, 0), (32000, 0), (32000, 50), (128256, 50), (777, 1), (64, 256)])
def test_sample_matches_oracle(V, top_k, dtype):
    B = 48
    ctx = specdec.Context(B, 1)
    logits, u, T = _case(B, V, dtype, seed=900 + V + top_k)
    tok = specdec.specdec_sample(ctx, specdec.from_numpy(logits), specdec.from_numpy(u), T, top_k)
    torch.cuda.synchronize()
    nb = _check(logits, u, T, top_k if 0 < top_k < V else None, tok.cpu().numpy())
    assert nb <= 1 and ctx.device_status() == 0
    ctx.close()


def test_sample_then_verify_against_itself_accepts_everything():
    """Tokens drafted by specdec_sample from q and verified against p = q are all accepted
    (Appendix C: ratio = 1 > r), and the call is repeatable."""
    B, V = 32, 32000
    ctx = specdec.Context(B, 1)
    logits, u, T = _case(B, V, "bf16", seed=77)
    lg = specdec.from_numpy(logits)
    tok = specdec.specdec_sample(ctx, lg, specdec.from_numpy(u), T)
    tok2 = specdec.specdec_sample(ctx, lg, specdec.from_numpy(u), T)
    assert torch.equal(tok, tok2)
    target = torch.stack([lg, lg], dim=1).contiguous()
    uni = specdec.from_numpy(np.ascontiguousarray(np.stack([u, u], axis=1)))
    n, _ = specdec.specdec_verify_correct(ctx, target, lg.view(B, 1, V), tok.view(B, 1), None, uni, T)
    torch.cuda.synchronize()
    assert torch.all(n == 1)
    ctx.close()


def test_sample_argument_errors():
    ctx = specdec.Context(4, 1)
    lg = torch.zeros(8, 16, device="cuda")
    u = torch.zeros(8, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_sample(ctx, lg, u, 1.0)
    assert e.value.code == specdec.EUNSUPPORTED
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_sample(ctx, lg[:4].contiguous(), u[:4].contiguous(), 0.0)
    assert e.value.code == specdec.EINVAL
    ctx.close()
