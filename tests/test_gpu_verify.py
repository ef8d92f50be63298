"""GPU parity of specdec_verify_correct / specdec_stop against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2405_19715_b200 import specdec, workloads as wl  # noqa: E402
from tests import parity  # noqa: E402
from oracle.specdec_oracle import stop_rule as orc_stop  # noqa: E402

KERNELS = [specdec.VERIFY_DIRECT, specdec.VERIFY_STREAM, specdec.VERIFY_FUSED, specdec.VERIFY_CLUSTER]
KERNEL_IDS = ["direct", "stream", "fused", "cluster"]


@pytest.fixture(scope="module")
def ctx():
    c = specdec.Context(max_B=256, max_K=32)
    yield c
    c.close()


def _stream_ok(inp):
    V = inp["target_logits"].shape[-1]
    es = 2 if inp["target_logits"].dtype == np.uint16 else 4
    return (V * es) % 16 == 0


def _random_problem(seed, B, K, V, dtype, T=1.0, sigma_n=1.0, ragged=True):
    cfg = wl.Workload(f"t{seed}", B=B, K=K, V=V, dtype=dtype, sigma_d=2.5, sigma_n=sigma_n, T=T, ragged=ragged, seed=seed)
    inp = wl.make_verify_inputs(cfg, threads=1)
    if ragged and B >= 3:        # make sure the degenerate lengths appear
        lens = inp["cand_len"].copy()
        lens[0], lens[1] = 0, K
        cfg2 = cfg
        inp = wl.make_verify_inputs(cfg2, threads=1)
        # re-poison consistently for the changed lengths by regenerating row by row
        for b in (0, 1):
            t, d, y = wl._row_logits(cfg, b, int(lens[b]), cfg.sigma_n, False)
            inp["target_logits"][b], inp["draft_logits"][b], inp["cand_tokens"][b] = t, d, y
        inp["cand_len"] = lens
    return inp


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 2, 7, 8, 33, 1000, 4104, 20000])
@pytest.mark.parametrize("K", [1, 2, 16])
def test_small_shapes(ctx, V, K, dtype, flags):
    inp = _random_problem(1000 + V + K, B=5, K=K, V=V, dtype=dtype, T=0.9)
    if flags in (specdec.VERIFY_STREAM, specdec.VERIFY_FUSED) and not _stream_ok(inp):
        pytest.skip("rows not 16-byte aligned: served by the direct kernel")
    gpu = parity.run_gpu_verify(ctx, inp, flags)
    rep = parity.classify_rows(inp, gpu, dtype="f32")      # bf16 inputs are widened exactly: same bar
    assert ctx.device_status() == 0
    assert rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == 5


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3"])
def test_configs_1_to_3(ctx, name, flags):
    cfg = wl.CONFIGS[name]
    inp = wl.make_verify_inputs(cfg)
    gpu = parity.run_gpu_verify(ctx, inp, flags)
    rep = parity.classify_rows(inp, gpu, dtype="f32")
    print(name, rep)
    assert ctx.device_status() == 0
    # the same call again must give bit-identical outputs (no order-dependent race)
    gpu2 = parity.run_gpu_verify(ctx, inp, flags)
    for k in ("n_accepted", "next_token", "accept_ratio", "row_stats", "resid_mass"):
        assert np.array_equal(gpu[k], gpu2[k]), k


@pytest.fixture(scope="module")
def cfg4_problem():
    """cfg4's inputs and the oracle's answer for every one of its 256 rows, made once for all kernels."""
    cfg = wl.CONFIGS["cfg4"]
    inp = wl.make_verify_inputs(cfg)
    return cfg, inp, parity.oracle_rows(inp)


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
def test_config4_full_size_every_row(ctx, cfg4_problem, flags):
    """Full-size cfg4 (B=256, K=16, V=128256, bf16) in the launch configuration the benchmark times:
    every row's n, y', accept ratios, p(y), q(y), normalisers and residual mass against the oracle."""
    cfg, inp, oracle_out = cfg4_problem
    gpu = parity.run_gpu_verify(ctx, inp, flags)
    assert ctx.device_status() == 0
    rep = parity.classify_rows(inp, gpu, dtype="f32", oracle_out=oracle_out)
    print("cfg4", KERNEL_IDS[KERNELS.index(flags)], rep)
    assert rep["rows"] == cfg.B and rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == cfg.B
    # rows whose drafted tokens carry +12 on the target are accepted almost surely
    peaked = np.nonzero(inp["peaked"])[0]
    assert (gpu["n_accepted"][peaked] == cfg.K).mean() > 0.8
    if flags == specdec.VERIFY_DIRECT:
        # the same launch with the early exit: identical n and y' on all 256 rows, and (7 waves, earliest
        # positions first) a large share of the logit rows left unread
        ctx.early_exit_count()
        fast = parity.run_gpu_verify(ctx, inp, flags | specdec.VERIFY_EARLY_EXIT, want_stats=False)
        unread = ctx.early_exit_count()
        assert ctx.device_status() == 0
        assert np.array_equal(fast["n_accepted"], gpu["n_accepted"]) and np.array_equal(fast["next_token"], gpu["next_token"])
        rows = int((2 * inp["cand_len"].astype(np.int64) + 1).sum())
        print("cfg4 early exit: logit rows not read", unread, "of", rows)
        assert rows // 4 < unread < rows


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
def test_special_cases(ctx, flags):
    rng = np.random.default_rng(3)
    B, K, V = 6, 5, 4096
    d = rng.normal(scale=3, size=(B, K, V)).astype(np.float32)
    t = np.concatenate([d, rng.normal(size=(B, 1, V)).astype(np.float32)], axis=1)
    y = rng.integers(0, V, size=(B, K)).astype(np.int32)
    u = wl.uniforms_24bit(rng, (B, K + 1))
    base = dict(target_logits=t, draft_logits=d, cand_tokens=y, cand_len=None, uniforms=u, temperature=np.float32(1.0))
    # identical models: everything accepted, bonus draw from p_{K+1}
    gpu = parity.run_gpu_verify(ctx, base, flags)
    assert np.all(gpu["n_accepted"] == K) and np.all(gpu["accept_ratio"] == 1.0)
    parity.classify_rows(base, gpu, dtype="f32")
    # very high temperature: both uniform
    hot = dict(base, target_logits=rng.normal(size=(B, K + 1, V)).astype(np.float32), temperature=np.float32(1e30))
    assert np.all(parity.run_gpu_verify(ctx, hot, flags)["n_accepted"] == K)
    # target one-hot on a token the draft did not pick: certain rejection, residual is a point mass
    t3 = t.copy()
    other = (y + 1) % V
    for b in range(B):
        t3[b, np.arange(K), other[b]] += 200.0
    peaked = dict(base, target_logits=t3)
    gpu = parity.run_gpu_verify(ctx, peaked, flags)
    assert np.all(gpu["n_accepted"] == 0) and np.array_equal(gpu["next_token"], other[:, 0])
    parity.classify_rows(peaked, gpu, dtype="f32")
    # masked (-inf) logits and huge offsets do not break the statistics
    t4, d4 = t.copy(), d.copy()
    t4[:, :, :100] = -np.inf
    d4[:, :, :100] = -np.inf
    t4[:, :, 100:] += 3.0e4
    y4 = np.maximum(y, 100).astype(np.int32)
    masked = dict(base, target_logits=t4, draft_logits=d4, cand_tokens=y4)
    gpu = parity.run_gpu_verify(ctx, masked, flags)
    parity.classify_rows(masked, gpu, dtype="f32")
    assert np.all(gpu["next_token"] >= 100)
    # a drafted token masked in both rows: p(y) = q(y) = 0 is a certain rejection, y' never lands on it
    t5, d5 = t + rng.normal(scale=0.8, size=t.shape).astype(np.float32), d.copy()
    for b in range(B):
        t5[b, 2, y[b, 2]] = d5[b, 2, y[b, 2]] = -np.inf
    u5 = u.copy()
    u5[:, :K] = 0.0                                                                    # r = 0 accepts any ratio > 0
    both = dict(base, target_logits=t5, draft_logits=d5, uniforms=u5)
    gpu = parity.run_gpu_verify(ctx, both, flags)
    assert np.all(gpu["n_accepted"] == 2) and np.all(gpu["accept_ratio"][:, 2] == 0.0)
    parity.classify_rows(both, gpu, dtype="f32")
    # low temperature approaches greedy decoding
    cold = dict(base, target_logits=t + rng.normal(scale=1.0, size=t.shape).astype(np.float32),
                cand_tokens=d.argmax(-1).astype(np.int32), temperature=np.float32(0.05))
    gpu = parity.run_gpu_verify(ctx, cold, flags)
    parity.classify_rows(cold, gpu, dtype="f32")


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
def test_outputs_ignore_positions_after_first_rejection(ctx, flags):
    cfg = wl.Workload("inv", B=16, K=8, V=8192, dtype="bf16", sigma_d=3.0, sigma_n=1.5, T=1.0, seed=77)
    inp = wl.make_verify_inputs(cfg)
    g1 = parity.run_gpu_verify(ctx, inp, flags)
    inp2 = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in inp.items()}
    rng = np.random.default_rng(1)
    for b in range(cfg.B):
        n = g1["n_accepted"][b]
        inp2["target_logits"][b, n + 1:] = wl.f32_to_bf16_bits(rng.normal(scale=9, size=inp2["target_logits"][b, n + 1:].shape).astype(np.float32))
        inp2["draft_logits"][b, n + 1:] = wl.f32_to_bf16_bits(rng.normal(scale=9, size=inp2["draft_logits"][b, n + 1:].shape).astype(np.float32))
        inp2["cand_tokens"][b, n + 1:] = (inp2["cand_tokens"][b, n + 1:] + 1) % cfg.V
    g2 = parity.run_gpu_verify(ctx, inp2, flags)
    assert np.array_equal(g1["n_accepted"], g2["n_accepted"]) and np.array_equal(g1["next_token"], g2["next_token"])


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
def test_bad_data_sets_status_without_trapping(ctx, flags):
    cfg = wl.Workload("bad", B=6, K=4, V=2048, dtype="bf16", sigma_d=3.0, sigma_n=1.0, T=1.0, seed=5)
    inp = wl.make_verify_inputs(cfg)
    inp["cand_len"] = np.array([4, 9, 4, -1, 4, 4], np.int32)
    inp["cand_tokens"][2, 1] = cfg.V
    inp["cand_tokens"][4, 0] = -3
    gpu = parity.run_gpu_verify(ctx, inp, flags)
    assert ctx.device_status() == (specdec.DATA_BAD_LENGTH | specdec.DATA_BAD_TOKEN)
    assert ctx.device_status() == 0                       # reading clears it
    for b in (1, 2, 3, 4):
        assert gpu["n_accepted"][b] == -1 and gpu["next_token"][b] == -1
    good = dict(inp, cand_len=np.array([4, 4, 4, 4, 4, 4], np.int32))
    rep = parity.classify_rows(good, gpu, rows=[0, 5], dtype="f32")
    assert rep["rows"] == 2
    # the context still works afterwards
    inp_ok = wl.make_verify_inputs(cfg)
    parity.classify_rows(inp_ok, parity.run_gpu_verify(ctx, inp_ok, flags), dtype="f32")


def test_argument_errors(ctx):
    t = torch.zeros(2, 3, 64, device="cuda")
    d = torch.zeros(2, 2, 64, device="cuda")
    y = torch.zeros(2, 2, dtype=torch.int32, device="cuda")
    u = torch.zeros(2, 3, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_verify_correct(ctx, t, d, y, None, u, 0.0)
    assert e.value.code == specdec.EINVAL
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_verify_correct(ctx, t, d, y, None, u, float("nan"))
    assert e.value.code == specdec.EINVAL
    big = torch.zeros(300, 3, 8, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_verify_correct(ctx, big, torch.zeros(300, 2, 8, device="cuda"),
                                       torch.zeros(300, 2, dtype=torch.int32, device="cuda"), None,
                                       torch.zeros(300, 3, device="cuda"), 1.0)
    assert e.value.code == specdec.EUNSUPPORTED
    with pytest.raises(specdec.SpecdecError) as e:   # 66 bf16 = 132 bytes per row: not 16-byte aligned
        specdec.specdec_verify_correct(ctx, torch.zeros(2, 3, 66, device="cuda", dtype=torch.bfloat16),
                                       torch.zeros(2, 2, 66, device="cuda", dtype=torch.bfloat16), y, None, u, 1.0,
                                       flags=specdec.VERIFY_STREAM)
    assert e.value.code == specdec.EUNSUPPORTED


def test_host_entry_point_matches_device_entry_point(ctx):
    cfg = wl.CONFIGS["cfg2"]
    inp = wl.make_verify_inputs(cfg)
    gpu = parity.run_gpu_verify(ctx, inp)
    h = {k: parity.to_torch(np.ascontiguousarray(inp[k]), "cpu", pin=True)
         for k in ("target_logits", "draft_logits", "cand_tokens", "cand_len", "uniforms")}
    ratio = torch.empty(cfg.B, cfg.K).pin_memory()
    n, tok = specdec.specdec_verify_correct_host(ctx, h["target_logits"], h["draft_logits"], h["cand_tokens"],
                                                 h["cand_len"], h["uniforms"], float(inp["temperature"]),
                                                 accept_ratio=ratio)
    assert np.array_equal(n.numpy(), gpu["n_accepted"]) and np.array_equal(tok.numpy(), gpu["next_token"])
    assert np.array_equal(ratio.numpy(), gpu["accept_ratio"])


def test_stop_rule_parity(ctx):
    for name, hs in (("cfg1", [0.5]), ("cfg3", [0.3, 0.5, 0.7])):
        cfg = wl.CONFIGS[name]
        a = wl.make_accept_prob(cfg)
        lens = wl.make_cand_len(cfg) if cfg.ragged else None
        ta = torch.from_numpy(a).cuda()
        tl = None if lens is None else torch.from_numpy(lens).cuda()
        for h in hs:
            pos = specdec.specdec_stop(ctx, ta, h, tl).cpu().numpy()
            rep = parity.classify_stop(a, h, pos, lens)
            assert rep["exact"] + rep["boundary"] == cfg.B
    # a candidate length outside [0, K] gives -1 for that row only and sets the status bit
    a = np.random.default_rng(2).uniform(0.5, 1.0, size=(5, 6)).astype(np.float32)
    lens = np.array([6, 7, 3, -1, 0], np.int32)
    pos = specdec.specdec_stop(ctx, torch.from_numpy(a).cuda(), 0.4, torch.from_numpy(lens).cuda()).cpu().numpy()
    assert ctx.device_status() == specdec.DATA_BAD_LENGTH and ctx.device_status() == 0
    assert pos[1] == -1 and pos[3] == -1
    good = [0, 2, 4]
    assert np.array_equal(pos[good], orc_stop(a[good], 0.4, lens[good]))
    # thresholds outside (0,1) and rows of ones
    a = np.ones((4, 7), np.float32)
    assert np.all(specdec.specdec_stop(ctx, torch.from_numpy(a).cuda(), 0.0).cpu().numpy() == 7)
    b = np.full((4, 7), 0.9, np.float32)
    assert np.all(specdec.specdec_stop(ctx, torch.from_numpy(b).cuda(), -0.5).cpu().numpy() == 0)
    assert np.all(specdec.specdec_stop(ctx, torch.from_numpy(b).cuda(), 1.0).cpu().numpy() == 7)
    big = np.random.default_rng(0).uniform(0.3, 1.0, size=(3000, 20)).astype(np.float32)
    pos = specdec.specdec_stop(specdec.Context(3000, 20), torch.from_numpy(big).cuda(), 0.6).cpu().numpy()
    rep = parity.classify_stop(big, 0.6, pos)
    assert rep["exact"] + rep["boundary"] == 3000


def test_bounded_wait_reports_and_context_survives(ctx):
    """A wait that can never complete ends by itself, sets the status bit, and leaves the context usable."""
    specdec.specdec_selftest_wait_limit(ctx)
    assert ctx.device_status() == specdec.DATA_WAIT_LIMIT
    assert ctx.device_status() == 0
    cfg = wl.CONFIGS["cfg2"]
    inp = wl.make_verify_inputs(cfg)
    for flags in KERNELS:
        parity.classify_rows(inp, parity.run_gpu_verify(ctx, inp, flags), dtype="f32")
    assert ctx.device_status() == 0


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
def test_wide_shapes(ctx, flags):
    """K = 32 (the ballot's full width), a batch larger than the SM count, a vocabulary of 262144."""
    for B, K, V, dtype in ((200, 32, 2048, "bf16"), (3, 2, 262144, "bf16"), (2, 3, 100000, "f32")):
        cfg = wl.Workload("wide", B=B, K=K, V=V, dtype=dtype, sigma_d=3.0, sigma_n=1.0, T=0.9, ragged=True, seed=B + V)
        inp = wl.make_verify_inputs(cfg)
        gpu = parity.run_gpu_verify(ctx, inp, flags)
        rep = parity.classify_rows(inp, gpu, dtype="f32")
        assert rep["rows"] == B and ctx.device_status() == 0


@pytest.mark.parametrize("flags", KERNELS, ids=KERNEL_IDS)
def test_many_candidates_per_row(flags):
    """K = 80: more positions than one ballot word or the fused kernel's six-bit row record hold."""
    c = specdec.Context(max_B=4, max_K=80)
    cfg = wl.Workload("k80", B=4, K=80, V=2048, dtype="bf16", sigma_d=2.0, sigma_n=0.3, T=1.0, ragged=True, seed=80)
    inp = wl.make_verify_inputs(cfg, threads=1)
    inp["cand_len"][:] = [80, 79, 33, 64]
    inp = dict(inp)
    # regenerate the rows for the forced lengths so that unread rows stay poisoned consistently
    for b in range(4):
        t, d, y = wl._row_logits(cfg, b, int(inp["cand_len"][b]), cfg.sigma_n, False)
        inp["target_logits"][b], inp["draft_logits"][b], inp["cand_tokens"][b] = t, d, y
    inp["draft_logits"][0] = inp["target_logits"][0][:80]      # p = q on row 0: all 80 candidates are accepted
    inp["draft_logits"][3, :40] = inp["target_logits"][3, :40]  # row 3 gets past the first ballot word at least
    gpu = parity.run_gpu_verify(c, inp, flags)
    rep = parity.classify_rows(inp, gpu, dtype="f32")
    assert rep["rows"] == 4 and c.device_status() == 0
    assert gpu["n_accepted"][0] == 80 and gpu["n_accepted"][3] >= 40
    c.close()


def test_gpu_draws_follow_the_target_law():
    """Secondary statistical check of the CUDA path itself: with one candidate per row drawn from q and
    seeded uniforms, the token a row emits (the candidate when accepted, y' otherwise) must be
    distributed as p (Appendix C).  2e5 rows at V = 8, chi-square with 7 degrees of freedom; the same
    rows also emit p-distributed bonus tokens when every candidate is accepted (checked on the rows
    that accept)."""
    rng = np.random.default_rng(99)
    V, N = 8, 200_000
    t = rng.normal(scale=1.5, size=V).astype(np.float32)
    d = rng.normal(scale=1.5, size=V).astype(np.float32)
    p = np.exp(t.astype(np.float64)); p /= p.sum()
    q = np.exp(d.astype(np.float64)); q /= q.sum()
    ys = rng.choice(V, size=N, p=q).astype(np.int32)
    uni = rng.random((N, 2)).astype(np.float32)
    uni = np.minimum(uni, np.float32(1.0 - 2.0 ** -24))
    big = specdec.Context(max_B=N, max_K=1)
    try:
        inp = dict(target_logits=np.broadcast_to(t, (N, 2, V)).copy(), draft_logits=np.broadcast_to(d, (N, 1, V)).copy(),
                   cand_tokens=ys.reshape(N, 1), cand_len=None, uniforms=uni, temperature=1.0)
        gpu = parity.run_gpu_verify(big, inp, specdec.VERIFY_DIRECT, want_stats=False)
        assert big.device_status() == 0
    finally:
        big.close()
    n, nxt = gpu["n_accepted"], gpu["next_token"]
    emitted = np.where(n == 1, ys, nxt)
    counts = np.bincount(emitted, minlength=V)
    chi2 = ((counts - N * p) ** 2 / (N * p)).sum()
    assert chi2 < 29.9, (chi2, counts)                      # P(chi2_7 > 29.9) ~ 1e-4
    # P(accept) = sum min(p, q)
    acc = float((n == 1).mean())
    assert abs(acc - np.minimum(p, q).sum()) < 4.0 * np.sqrt(0.25 / N)
    # the bonus token of the accepting rows (target row 1 = the same p) is p-distributed too
    bonus = nxt[n == 1]
    cb = np.bincount(bonus, minlength=V)
    chi2b = ((cb - len(bonus) * p) ** 2 / (len(bonus) * p)).sum()
    assert chi2b < 29.9, (chi2b, cb)


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg5"])
def test_early_exit_leaves_the_outputs_unchanged(name):
    """SPECDEC_VERIFY_EARLY_EXIT: units that start after an earlier position of their row has been rejected
    read nothing.  n_accepted and next_token must be what the oracle says (and what the call without the bit
    gives), bad tokens after the first rejection must still be reported, and on a batch of several waves a
    good share of the units must indeed have left early."""
    cfg = wl.CONFIGS[name]
    inp = wl.make_verify_inputs(cfg)
    c = specdec.Context(cfg.B, cfg.K)
    try:
        base = parity.run_gpu_verify(c, inp, specdec.VERIFY_DIRECT, want_stats=False)
        c.early_exit_count()
        fast = parity.run_gpu_verify(c, inp, specdec.VERIFY_DIRECT | specdec.VERIFY_EARLY_EXIT, want_stats=False)
        left = c.early_exit_count()
        assert c.device_status() == 0
        assert np.array_equal(base["n_accepted"], fast["n_accepted"])
        assert np.array_equal(base["next_token"], fast["next_token"])
        rep = parity.classify_rows(inp, fast, dtype="f32", check_probs=False)
        assert rep["exact"] + rep["boundary_n"] + rep["boundary_token"] == cfg.B
        units = int((inp["cand_len"].astype(np.int64) + 1).sum())
        rows = int((2 * inp["cand_len"].astype(np.int64) + 1).sum())
        print(name, "units", units, "logit rows", rows, "rows not read", left)
        assert 0 <= left < rows
        if name == "cfg5":
            assert left > rows // 4                   # 3.7 waves, earliest positions first
        # with the optional outputs requested the bit is ignored: all positions are computed
        full = parity.run_gpu_verify(c, inp, specdec.VERIFY_DIRECT | specdec.VERIFY_EARLY_EXIT, want_stats=True)
        assert c.early_exit_count() == 0
        parity.classify_rows(inp, full, dtype="f32")
        # a bad token behind the first rejection is still seen
        bad = dict(inp)
        bad["cand_tokens"] = inp["cand_tokens"].copy()
        b = int(np.argmax((base["n_accepted"] + 1 < inp["cand_len"])))      # a row with a position after its first rejection
        if base["n_accepted"][b] + 1 < inp["cand_len"][b]:
            bad["cand_tokens"][b, inp["cand_len"][b] - 1] = cfg.V + 5
            out = parity.run_gpu_verify(c, bad, specdec.VERIFY_DIRECT | specdec.VERIFY_EARLY_EXIT, want_stats=False)
            assert c.device_status() & specdec.DATA_BAD_TOKEN
            assert out["n_accepted"][b] == -1 and out["next_token"][b] == -1
    finally:
        c.close()
