"""specdec_verify_correct_static: the entry point for callers that are not allowed to allocate
device memory (a server whose memory pool owns the whole GPU, a plugin that must not call
cudaMalloc after start-up).  It has to give the same answers as the context-based entry point,
call after call, although all its calls share one fixed scratch array that is never reset between
them by the caller.  Collected last on purpose: a failure here cannot hide the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2405_19715_b200 import specdec, workloads as wl  # noqa: E402


def _device_inputs(cfg):
    inp = wl.make_verify_inputs(cfg)
    dev = {k: specdec.from_numpy(inp[k]) for k in ("target_logits", "draft_logits", "cand_tokens", "cand_len", "uniforms")}
    return inp, dev


def _reference(cfg, dev, T):
    ctx = specdec.Context(cfg.B, cfg.K)
    n, t = specdec.specdec_verify_correct(ctx, dev["target_logits"], dev["draft_logits"], dev["cand_tokens"],
                                          dev["cand_len"], dev["uniforms"], T, flags=specdec.VERIFY_DIRECT)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    out = n.cpu().numpy(), t.cpu().numpy()
    ctx.close()
    return out


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    """Two different problems, one after the other on the same stream: the second call finds the
    first call's flags, draws and counters in the shared array and must not be confused by them.
    Discrete outputs are compared exactly (both paths run the same fp32 arithmetic)."""
    cfg_a = wl.CONFIGS["cfg3"]                                   # ragged lengths, bf16
    cfg_b = wl.Workload("static_b", B=40, K=12, V=8000, dtype="f32", sigma_d=3.0, sigma_n=1.2, T=0.8, ragged=True,
                        seed=991)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for cfg in (cfg_a, cfg_b, cfg_a):
        inp, dev = _device_inputs(cfg)
        T = float(inp["temperature"])
        want_n, want_t = _reference(cfg, dev, T)
        n = torch.full((cfg.B,), -9, dtype=torch.int32, device="cuda")
        t = torch.full((cfg.B,), -9, dtype=torch.int32, device="cuda")
        for _ in range(2):                                        # the same problem twice as well
            n.fill_(-9)
            t.fill_(-9)
            specdec.specdec_verify_correct_static(dev["target_logits"], dev["draft_logits"], dev["cand_tokens"],
                                                  dev["cand_len"], dev["uniforms"], T, n, t, data_status=status)
            torch.cuda.synchronize()
            assert np.array_equal(n.cpu().numpy(), want_n)
            assert np.array_equal(t.cpu().numpy(), want_t)
    assert int(status.item()) == 0


def test_static_entry_point_rejects_oversized_problems():
    B, K = 2048, 8                                                # 2048 * 9 = 18432 units > 16384
    z = torch.zeros(1, device="cuda")
    t = torch.zeros((B, K + 1, 8), device="cuda")
    d = torch.zeros((B, K, 8), device="cuda")
    y = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    u = torch.zeros((B, K + 1), device="cuda")
    n = torch.zeros(B, dtype=torch.int32, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_verify_correct_static(t, d, y, None, u, 1.0, n, n.clone())
    assert e.value.code == specdec.EUNSUPPORTED and "16384" in str(e.value)
    del z
