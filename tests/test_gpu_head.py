"""GPU parity of specdec_accept_head (tcgen05 GEMMs) and of the head -> stop -> verify chain of
cfg5 against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import specdec_oracle as orc  # noqa: E402
from paper_2405_19715_b200 import specdec, workloads as wl  # noqa: E402
from tests import parity  # noqa: E402

HEAD_RTOL = 2e-2      # tolerance for head outputs computed from bf16 activations


def _head_problem(seed, B, K, d, depth, with_bias, std=0.05):
    rng = np.random.default_rng(seed)
    hidden = wl.f32_to_bf16_bits(rng.standard_normal((B, K, d), dtype=np.float32))
    Ws = [wl.f32_to_bf16_bits((rng.standard_normal((d, d), dtype=np.float32) * std)) for _ in range(depth)]
    bs = [wl.f32_to_bf16_bits(rng.standard_normal(d, dtype=np.float32) * 0.3) if with_bias else None for _ in range(depth)]
    w_out = wl.f32_to_bf16_bits(rng.standard_normal(d, dtype=np.float32) * std)
    return hidden, Ws, bs, w_out, float(rng.normal() * 0.2)


def _run_head(ctx, hidden, Ws, bs, w_out, b_out):
    th = specdec.from_numpy(hidden)
    tW = [specdec.from_numpy(w) for w in Ws]
    tb = [None if b is None else specdec.from_numpy(b) for b in bs]
    out = specdec.specdec_accept_head(ctx, th, tW, tb, specdec.from_numpy(w_out), b_out)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return out.cpu().numpy()


@pytest.mark.parametrize("d", [128, 256, 384, 512])
@pytest.mark.parametrize("depth", [0, 1, 2, 3])
@pytest.mark.parametrize("with_bias", [False, True])
@pytest.mark.parametrize("rows", [(7, 23), (9, 33)], ids=["161rows", "297rows"])
def test_head_small_shapes(d, depth, with_bias, rows):
    B, K = rows                       # 161 rows use the weights-as-M kernel, 297 rows the 128 x 128/256 tiles;
                                      # both leave a ragged last row tile
    ctx = specdec.Context(B, K, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(100 + d + depth, B, K, d, depth, with_bias)
    got = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
    want = orc.accept_head(hidden, list(zip(Ws, bs)), w_out, b_out)
    err = np.abs(got - want) / want
    assert err.max() <= HEAD_RTOL, (err.max(), got.ravel()[:4], want.ravel()[:4])
    # a transposed or mis-tiled operand would be off by far more than the tolerance; make sure the
    # outputs are not degenerate either
    assert want.std() > 1e-3
    ctx.close()


@pytest.mark.parametrize("rows,d,depth", [((13, 47), 256, 1), ((13, 47), 512, 2), ((25, 31), 768, 2), ((64, 16), 1024, 3),
                                          ((30, 20), 512, 8), ((80, 42), 768, 4), ((60, 42), 1024, 5)],
                         ids=["611x256", "611x512", "775x768", "1024x1024", "600x512x8", "3360x768x4", "2520x1024x5"])
def test_head_many_row_tiles(rows, d, depth):
    """Several row tiles with a ragged last one, widths up to 1024 and depth up to 8.  All blocks of a call are
    tiles of one launch, a block's tiles waiting for the row block they read: the last two cases have 168 and
    200 tiles of 256 x 256 (a pair of CTAs each; the smaller cases get 128-wide tiles), so every pair gets two or
    three of them, from different blocks (the double-buffered accumulator and the stage ring across tiles and
    blocks); depth 4 and more re-use the two activation buffers within the launch.  The call is repeatable bit
    for bit."""
    B, K = rows
    ctx = specdec.Context(B, K, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(300 + d + depth, B, K, d, depth, True, std=0.02)
    got = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
    want = orc.accept_head(hidden, list(zip(Ws, bs)), w_out, b_out)
    err = np.abs(got - want) / want
    assert err.max() <= HEAD_RTOL, (err.max(), np.argmax(err), got.ravel()[:4], want.ravel()[:4])
    assert want.std() > 1e-3
    got2 = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
    assert np.array_equal(got, got2)
    ctx.close()



@pytest.mark.parametrize("rows,d,depth", [((30, 20), 384, 3), ((80, 42), 768, 4), ((9, 33), 512, 2)],
                         ids=["600x384x3", "3360x768x4", "297x512x2"])
def test_head_launch_forms_agree(rows, d, depth):
    """The three forms specdec_accept_head falls back through for more than 256 rows -- pairs of CTAs in one
    cooperative launch, one CTA per tile in one cooperative launch, one launch per block (with and without
    pairs) -- each against the oracle and against one another (the arithmetic per output is the same)."""
    B, K = rows
    ctx = specdec.Context(B, K, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(900 + d + depth, B, K, d, depth, True, std=0.02)
    want = orc.accept_head(hidden, list(zip(Ws, bs)), w_out, b_out)
    outs = {}
    for pair in (True, False):
        for coop in (True, False):
            ctx.head_launch_mode(pair=pair, cooperative=coop)
            n0 = ctx.launch_count()
            got = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
            assert ctx.launch_count() - n0 == (1 if coop else depth), (pair, coop)
            err = np.abs(got - want) / want
            assert err.max() <= HEAD_RTOL, (pair, coop, err.max())
            outs[(pair, coop)] = got
    ref = outs[(True, True)]
    for key, got in outs.items():
        np.testing.assert_allclose(got, ref, rtol=1e-5, atol=0, err_msg=str(key))
    ctx.close()


@pytest.mark.parametrize("rows", [(3, 20), (25, 31)], ids=["60rows", "775rows"])
def test_head_call_replayed_from_a_graph(rows):
    """One captured call replayed three times in a row gives the eager call's bits every time: whatever the
    kernels count in the context's scratch is back to its initial state when a call ends."""
    B, K = rows
    d, depth = 512, 3
    ctx = specdec.Context(B, K, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(1200 + B, B, K, d, depth, True, std=0.02)
    th, tw = specdec.from_numpy(hidden), specdec.from_numpy(w_out)
    tW = [specdec.from_numpy(w) for w in Ws]
    tb = [specdec.from_numpy(b) for b in bs]
    out = torch.empty(B, K, dtype=torch.float32, device="cuda")
    specdec.specdec_accept_head(ctx, th, tW, tb, tw, b_out, out)
    torch.cuda.synchronize()
    want = out.clone()
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=s):
        specdec.specdec_accept_head(ctx, th, tW, tb, tw, b_out, out)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, want)
    assert ctx.device_status() == 0
    ctx.close()

@pytest.mark.parametrize("rows", [1, 2, 3, 4, 5, 8, 9, 13, 16, 17, 32, 33, 64, 65])
@pytest.mark.parametrize("d,depth,with_bias", [(256, 1, True), (512, 3, False), (4096, 2, True)])
def test_head_few_rows(rows, d, depth, with_bias):
    """One drafted token for 1 to 65 sequences (the weights-as-M kernel): row counts that are not multiples of
    16 leave zero-padded accumulator columns; d = 256 splits the reduction over 4 CTAs of 1 k-block each,
    d = 4096 of 16."""
    ctx = specdec.Context(rows, 1, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(700 + rows + d, rows, 1, d, depth, with_bias, std=0.02 if d > 512 else 0.05)
    got = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
    want = orc.accept_head(hidden, list(zip(Ws, bs)), w_out, b_out)
    err = np.abs(got - want) / want
    assert err.max() <= HEAD_RTOL, (err.max(), got.ravel()[:4], want.ravel()[:4])
    assert np.array_equal(got, _run_head(ctx, hidden, Ws, bs, w_out, b_out))
    ctx.close()


def test_head_reduces_to_logistic_regression_when_weights_are_zero():
    B, K, d = 4, 40, 256
    ctx = specdec.Context(B, K, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(5, B, K, d, 2, False)
    Ws = [np.zeros_like(w) for w in Ws]
    got = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
    want = orc.accept_head(hidden, [], w_out, b_out)
    np.testing.assert_allclose(got, want, rtol=1e-4)
    ctx.close()


def test_head_argument_errors():
    ctx = specdec.Context(4, 4, max_d=256)
    h = torch.zeros(4, 4, 192, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(192, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_accept_head(ctx, h, [], None, w, 0.0)
    assert e.value.code == specdec.EUNSUPPORTED
    h = torch.zeros(4, 4, 512, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(specdec.SpecdecError) as e:
        specdec.specdec_accept_head(ctx, h, [], None, torch.zeros(512, dtype=torch.bfloat16, device="cuda"), 0.0)
    assert e.value.code == specdec.EUNSUPPORTED
    ctx.close()


def test_config5_head_stop_verify_chain():
    """cfg5: hidden [128,16,4096] -> D=2 head -> stop at h=0.5 -> cand_len = min(stop_pos + 2, K)
    -> verify/correct at V=32000 (bf16, T=0.7)."""
    cfg = wl.CONFIGS["cfg5"]
    ctx = specdec.Context(cfg.B, cfg.K, max_d=cfg.d)
    hd = wl.make_head_inputs(cfg)
    Ws = [w for w, _ in hd["blocks"]]
    bs = [b for _, b in hd["blocks"]]
    got = _run_head(ctx, hd["hidden"], Ws, bs, hd["w_out"], float(hd["b_out"]))
    want = orc.accept_head(hd["hidden"], hd["blocks"], hd["w_out"], float(hd["b_out"]))
    err = np.abs(got - want) / want
    print("cfg5 head max rel err", err.max())
    assert err.max() <= HEAD_RTOL
    # stop rule on the GPU's own probabilities (same inputs on both sides)
    pos = specdec.specdec_stop(ctx, torch.from_numpy(got).cuda(), cfg.h).cpu().numpy()
    rep = parity.classify_stop(got, cfg.h, pos)
    assert rep["exact"] + rep["boundary"] == cfg.B
    cand_len = np.minimum(pos + 2, cfg.K).astype(np.int32)     # Algorithm 1: one more token was drafted
    print("cfg5 cand_len histogram", np.bincount(cand_len, minlength=cfg.K + 1).tolist())
    inp = wl.make_verify_inputs(cfg)
    inp["cand_len"] = cand_len
    gpu = parity.run_gpu_verify(ctx, inp)
    rep = parity.classify_rows(inp, gpu, dtype="f32")
    print("cfg5 verify", rep)
    assert ctx.device_status() == 0
    ctx.close()


def test_head_at_the_benchmark_shape():
    """The shape the benchmark times: B*K = 4096 rows (cfg4's 256 x 16 positions), d = 4096, D = 2 of
    the cfg5 recipe, i.e. 512 tiles of 128 x 256 on 148 persistent CTAs (3.46 tiles per CTA).  All 4096
    outputs against the oracle; repeatable bit for bit."""
    cfg = wl.CONFIGS["cfg5"].scaled(B=256, K=16)
    ctx = specdec.Context(cfg.B, cfg.K, max_d=cfg.d)
    hd = wl.make_head_inputs(cfg)
    Ws = [w for w, _ in hd["blocks"]]
    bs = [b for _, b in hd["blocks"]]
    got = _run_head(ctx, hd["hidden"], Ws, bs, hd["w_out"], float(hd["b_out"]))
    want = orc.accept_head(hd["hidden"], hd["blocks"], hd["w_out"], float(hd["b_out"]))
    err = np.abs(got - want) / want
    print("head 4096 x 4096 x 2 max rel err", err.max())
    assert got.shape == (256, 16) and err.max() <= HEAD_RTOL and want.std() > 1e-2
    assert np.array_equal(got, _run_head(ctx, hd["hidden"], Ws, bs, hd["w_out"], float(hd["b_out"])))
    ctx.close()


@pytest.mark.parametrize("rows", [17, 32, 33, 64, 65, 128, 129, 200, 256])
def test_head_up_to_256_rows_at_full_width(rows):
    """17 to 256 rows at d = 4096, D = 2 (Eq. 3 once per drafted token for that many sequences)."""
    ctx = specdec.Context(rows, 1, max_d=4096)
    hidden, Ws, bs, w_out, b_out = _head_problem(900 + rows, rows, 1, 4096, 2, True, std=0.02)
    got = _run_head(ctx, hidden, Ws, bs, w_out, b_out)
    want = orc.accept_head(hidden, list(zip(Ws, bs)), w_out, b_out)
    err = np.abs(got - want) / want
    assert err.max() <= HEAD_RTOL, (err.max(), np.argmax(err))
    assert np.array_equal(got, _run_head(ctx, hidden, Ws, bs, w_out, b_out))
    ctx.close()


def test_online_head_and_stop_step_replay_algorithm_1():
    """Algorithm 1's loop, one drafted token per call: head on [B,1,d] (weights-as-M kernel), then
    specdec_stop_step.  Each step is checked against the oracle; the replay must also reproduce the
    batched head + stop rule."""
    B, K, d = 96, 6, 512
    ctx = specdec.Context(B, K, max_d=d)
    hidden, Ws, bs, w_out, b_out = _head_problem(77, B, K, d, 2, True, std=0.03)
    batched = _run_head(ctx, hidden, Ws, bs, w_out, b_out)                      # [B, K]
    tW = [specdec.from_numpy(w) for w in Ws]
    tb = [specdec.from_numpy(b) for b in bs]
    tw = specdec.from_numpy(w_out)
    h = 0.5
    p_hat = torch.ones(B, dtype=torch.float32, device="cuda")
    o_hat = np.ones(B)
    first = np.full(B, K)
    for j in range(K):
        step_hidden = np.ascontiguousarray(hidden[:, j:j + 1, :])
        a = specdec.specdec_accept_head(ctx, specdec.from_numpy(step_hidden), tW, tb, tw, b_out)   # [B, 1]
        want = orc.accept_head(step_hidden, list(zip(Ws, bs)), w_out, b_out)
        got = a.cpu().numpy()
        assert np.max(np.abs(got - want) / want) <= HEAD_RTOL
        np.testing.assert_allclose(got[:, 0], batched[:, j], rtol=1e-3)   # two kernels, two summation orders, bf16 activations
        stop = specdec.specdec_stop_step(ctx, a.reshape(B), p_hat, h).cpu().numpy()
        o_hat, o_stop = orc.stop_step(o_hat.astype(np.float32), got[:, 0], h)
        near = np.abs(1.0 - o_hat - np.float32(h)) < parity.BOUNDARY
        assert np.array_equal(stop[~near].astype(bool), o_stop[~near])
        np.testing.assert_allclose(p_hat.cpu().numpy(), o_hat, rtol=1e-6)
        first = np.where((first == K) & (stop == 1), j, first)
    pos = specdec.specdec_stop(ctx, torch.from_numpy(batched).cuda(), h).cpu().numpy()
    rep = parity.classify_stop(batched, h, pos)
    assert rep["exact"] + rep["boundary"] == B
    assert (first == pos).mean() > 0.95          # identical except where a product sits on the threshold
    assert ctx.device_status() == 0
    ctx.close()
