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
from tests import parity  # noqa: E402

KEYS = ("target_logits", "draft_logits", "cand_tokens", "cand_len", "uniforms")


def _device_inputs(inp):
    return {k: (None if inp.get(k) is None else specdec.from_numpy(inp[k])) for k in KEYS}


def _context_entry_point(cfg, dev, T):
    ctx = specdec.Context(cfg.B, cfg.K)
    n, t = specdec.specdec_verify_correct(ctx, dev["target_logits"], dev["draft_logits"], dev["cand_tokens"],
                                          dev["cand_len"], dev["uniforms"], T, flags=specdec.VERIFY_DIRECT)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    out = dict(n_accepted=n.cpu().numpy(), next_token=t.cpu().numpy())
    ctx.close()
    return out


def _static_call(dev, T, B, status):
    n = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    t = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    specdec.specdec_verify_correct_static(dev["target_logits"], dev["draft_logits"], dev["cand_tokens"],
                                          dev["cand_len"], dev["uniforms"], T, n, t, data_status=status)
    torch.cuda.synchronize()
    return dict(n_accepted=n.cpu().numpy(), next_token=t.cpu().numpy())


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    """Different problems one after the other on the same stream, each twice: a call finds the
    previous call's flags, draws and counters in the shared array and must not be confused by them.
    Every row is classified against the CPU oracle (exact, or within 1e-6 of a ratio / CDF boundary,
    the tolerance of the other verify tests), and compared with the context-based entry point,
    whose rows may differ from the static ones only where the oracle calls a boundary."""
    problems = [
        wl.CONFIGS["cfg3"],                                                                    # ragged lengths, bf16
        wl.Workload("static_b", B=40, K=12, V=8000, dtype="f32", sigma_d=3.0, sigma_n=1.2, T=0.8, ragged=True, seed=991),
        wl.Workload("static_c", B=7, K=5, V=4099, dtype="bf16", sigma_d=2.5, sigma_n=1.0, T=1.1, seed=17),   # rows not 16-byte aligned
        wl.Workload("static_d", B=6, K=3, V=1001, dtype="f32", sigma_d=2.5, sigma_n=0.8, T=1.0, seed=18),    # odd V, cand_len = NULL
        wl.CONFIGS["cfg3"],
    ]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    totals = dict(rows=0, exact=0, boundary=0, differs_from_context=0)
    for cfg in problems:
        inp = wl.make_verify_inputs(cfg)
        if cfg.name == "static_d":
            inp["cand_len"] = None
        dev = _device_inputs(inp)
        T = float(inp["temperature"])
        oracle_out = parity.oracle_rows(inp)
        want = _context_entry_point(cfg, dev, T)
        rep_want = parity.classify_rows(inp, want, dtype="f32", check_probs=False, oracle_out=oracle_out)
        for _ in range(2):                                        # the same problem twice as well
            got = _static_call(dev, T, cfg.B, status)
            rep = parity.classify_rows(inp, got, dtype="f32", check_probs=False, oracle_out=oracle_out)
            assert rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == cfg.B
            differs = (got["n_accepted"] != want["n_accepted"]) | (got["next_token"] != want["next_token"])
            assert differs.sum() <= sum(r[k] for r in (rep, rep_want) for k in ("boundary_n", "boundary_token"))
            totals["rows"] += cfg.B
            totals["exact"] += rep["exact"]
            totals["boundary"] += rep["boundary_n"] + rep["boundary_token"]
            totals["differs_from_context"] += int(differs.sum())
    print("static entry point", totals)
    assert int(status.item()) == 0


def test_static_entry_point_reports_bad_lengths_and_tokens_through_data_status():
    """A length outside [0, K] and tokens outside [0, V) give -1 for their rows and set the caller's
    status word; the good rows of the same call still match the oracle, and so does the next call."""
    cfg = wl.Workload("static_bad", B=6, K=4, V=2048, dtype="bf16", sigma_d=3.0, sigma_n=1.0, T=1.0, seed=5)
    inp = wl.make_verify_inputs(cfg)
    inp["cand_len"] = np.array([4, 9, 4, -1, 4, 4], np.int32)
    inp["cand_tokens"][2, 1] = cfg.V
    inp["cand_tokens"][4, 0] = -3
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = _static_call(_device_inputs(inp), 1.0, cfg.B, status)
    assert int(status.item()) == (specdec.DATA_BAD_LENGTH | specdec.DATA_BAD_TOKEN)
    for b in (1, 2, 3, 4):
        assert got["n_accepted"][b] == -1 and got["next_token"][b] == -1
    good = dict(inp, cand_len=np.array([4, 4, 4, 4, 4, 4], np.int32))
    assert parity.classify_rows(good, got, rows=[0, 5], dtype="f32", check_probs=False)["rows"] == 2
    status.zero_()
    clean = wl.make_verify_inputs(cfg)
    got = _static_call(_device_inputs(clean), 1.0, cfg.B, status)
    parity.classify_rows(clean, got, dtype="f32", check_probs=False)
    assert int(status.item()) == 0


def test_static_entry_point_rejects_oversized_problems():
    B, K = 2048, 8                                                # 2048 * 9 = 18432 units > 16384
    t = torch.zeros((B, K + 1, 8), device="cuda")
    d = torch.zeros((B, K, 8), device="cuda")
    y = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    u = torch.zeros((B, K + 1), device="cuda")
    n = torch.zeros(B, dtype=torch.int32, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_verify_correct_static(t, d, y, None, u, 1.0, n, n.clone())
    assert e.value.code == specdec.EUNSUPPORTED and "16384" in str(e.value)
