"""Pins for the CPU oracle: each check ties an oracle function to something fixed by the
paper or by mathematics (exact-rational brute force, closed forms, invariants, special
cases that reduce to an independent library routine, hand-worked fixtures), never to the
oracle's own formula retyped.  No GPU needed.
"""
from fractions import Fraction as Fr
from itertools import product
from pathlib import Path

import numpy as np
import pytest
import scipy.special
import torch

from oracle import specdec_oracle as orc

GOLDEN = Path(__file__).parent / "golden"


def frac_array(vals):
    a = np.empty(len(vals), dtype=object)
    a[:] = [Fr(v) for v in vals]
    return a


def simplex_grid(V, denom):
    """All probability vectors with entries k/denom, k >= 1."""
    for ks in product(range(1, denom), repeat=V - 1):
        last = denom - sum(ks)
        if last >= 1:
            yield frac_array([Fr(k, denom) for k in ks] + [Fr(last, denom)])


# ----------------------------------------------------------------------------- fixtures
def _parse_fixture(name):
    rows = []
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        rows.append([c.strip() for c in line.split("|")])
    return rows


@pytest.mark.parametrize("row", _parse_fixture("rejection_step_worked.txt"), ids=lambda r: r[0])
def test_worked_rejection_steps(row):
    """Appendix C rejection step, hand-worked values (tests/golden/rejection_step_worked.txt)."""
    _, p, q, y, r, u, acc, tok = row
    p, q = frac_array(p.split()), frac_array(q.split())
    y, r, u = int(y), Fr(r), Fr(u)
    # One candidate (L=1).  Row 1 of the target is a point mass on token 0 so the bonus
    # draw cannot be confused with the emitted first token.
    bonus = frac_array([1] + [0] * (len(p) - 1))
    n, nxt, ratios, _ = orc.verify_from_probs([p, bonus], [q], [y], 1, [r], u)
    assert n == int(acc)
    emitted = y if n == 1 else nxt
    assert emitted == int(tok)
    if n == 0:   # float64 path agrees away from exact ties
        pf, qf = p.astype(float), q.astype(float)
        if r != ratios[0]:
            n2, nxt2, _, _ = orc.verify_from_probs([pf, bonus.astype(float)], [qf], [y], 1, [float(r)], float(u) + 1e-12)
            assert (n2, nxt2) == (n, nxt)


@pytest.mark.parametrize("row", _parse_fixture("stop_rule_worked.txt"), ids=lambda r: r[0])
def test_worked_stop_rule(row):
    """Section 4.3 threshold rule, hand-worked dyadic values (tests/golden/stop_rule_worked.txt)."""
    _, a, h, want = row
    a = np.array([[float(x) for x in a.split()]], dtype=np.float32)
    got = orc.stop_rule(a, float(h))[0]
    assert got == (a.shape[1] if want == "none" else int(want))


# ----------------------------------------------------------------------------- exact law, one step
def _emitted_law_one_step(p, q, denom_grid):
    """Exact law of the token emitted at position 0 when y ~ q, r and u uniform.

    Every breakpoint of the accept test (p_y/q_y) and of the residual CDF is a multiple of
    1/denom_grid (the probabilities are multiples of 1/denom with denom_grid = lcm(1..denom)),
    so the midpoint rule over cells of width 1/denom_grid integrates the oracle exactly.
    """
    V = len(p)
    law = [Fr(0)] * V
    cell = Fr(1, denom_grid)
    mids = [Fr(2 * k + 1, 2 * denom_grid) for k in range(denom_grid)]
    bonus = frac_array([1] + [0] * (V - 1))
    for y in range(V):
        for r in mids:
            n, _, _, _ = orc.verify_from_probs([p, bonus], [q], [y], 1, [r], Fr(1, 2))
            if n == 1:
                law[y] += q[y] * cell
            else:
                for u in mids:
                    _, tok, _, _ = orc.verify_from_probs([p, bonus], [q], [y], 1, [r], u)
                    law[tok] += q[y] * cell * cell
    return law


def test_rejection_sampling_is_unbiased_exact():
    """Appendix C: the emitted token is distributed exactly as p (brute force, V<=4, exact rationals)."""
    count = 0
    for V, denom, grid in ((2, 6, 60), (3, 5, 60), (4, 5, 60)):
        pairs = list(simplex_grid(V, denom))
        step = max(1, len(pairs) // 6)
        for p in pairs[::step]:
            for q in pairs[1::step]:
                law = _emitted_law_one_step(p, q, grid)
                assert all(law[x] == p[x] for x in range(V)), (p, q, law)
                count += 1
    assert count >= 30


def test_acceptance_probability_and_residual_identities_exact():
    """P(accept) = sum_v min(p,q); residual mass = 1 - sum min(p,q) = TV(p,q); support only where p>q."""
    for V, denom in ((3, 7), (5, 8), (8, 11)):
        pairs = list(simplex_grid(V, denom))
        rng = np.random.default_rng(V)
        for _ in range(40):
            p = pairs[rng.integers(len(pairs))]
            q = pairs[rng.integers(len(pairs))]
            p_acc = sum(q[y] * min(Fr(1), orc.accept_ratio(p[y], q[y])) for y in range(V))
            overlap = sum(min(a, b) for a, b in zip(p, q))
            assert p_acc == overlap
            w = orc.residual(p, q)
            W = sum(w)
            assert W == 1 - overlap == sum(abs(a - b) for a, b in zip(p, q)) / 2
            assert all((w[v] == 0) == (p[v] <= q[v]) for v in range(V))
            assert all(w[v] == p[v] - q[v] for v in range(V) if p[v] > q[v])


def test_boundaries_exact():
    """r == ratio rejects (Algorithm 2 writes r >= p/q); token j owns [F_{j-1}, F_j)."""
    p, q = frac_array(["1/10", "1/5", "3/10", "2/5"]), frac_array(["2/5", "3/10", "1/5", "1/10"])
    bonus = frac_array([0, 0, 0, 1])
    eps = Fr(1, 10**12)
    assert orc.verify_from_probs([p, bonus], [q], [0], 1, [Fr(1, 4)], Fr(0))[0] == 0
    assert orc.verify_from_probs([p, bonus], [q], [0], 1, [Fr(1, 4) - eps], Fr(0))[0] == 1
    # residual CDF is (0, 0, 1/4, 1)
    for u, tok in ((Fr(0), 2), (Fr(1, 4) - eps, 2), (Fr(1, 4), 3), (1 - eps, 3)):
        assert orc.verify_from_probs([p, bonus], [q], [0], 1, [Fr(1, 2)], u)[1] == tok
    # ratio >= 1 always accepts because r < 1
    assert orc.verify_from_probs([p, bonus], [q], [3], 1, [1 - eps], Fr(0))[0] == 1


# ----------------------------------------------------------------------------- chained steps
def _chained_law_check(V, G, choices, trials, seed):
    """K=2 brute force.  Every acceptance ratio below 1 and every CDF breakpoint that the chosen
    probability vectors can produce is a multiple of 1/G, so midpoints of a 1/G grid integrate
    (r1, r2, u) exactly."""
    K = 2
    rng = np.random.default_rng(seed)

    def table():       # distribution after each history of length 0..K
        return {h: choices[rng.integers(len(choices))] for L in range(K + 1) for h in product(range(V), repeat=L)}

    for _ in range(trials):
        P, Q = table(), table()
        mids = [Fr(2 * k + 1, 2 * G) for k in range(G)]
        cell = Fr(1, G)
        law = {s: Fr(0) for s in product(range(V), repeat=K + 1)}
        exp_n = Fr(0)
        for ys in product(range(V), repeat=K):
            wq = Q[()][ys[0]] * Q[(ys[0],)][ys[1]]
            p_rows = [P[()], P[(ys[0],)], P[ys]]
            q_rows = [Q[()], Q[(ys[0],)]]
            for r1, r2, u in product(mids, repeat=3):
                n, nxt, _, _ = orc.verify_from_probs(p_rows, q_rows, list(ys), K, [r1, r2], u)
                out = tuple(ys[:n]) + (nxt,)
                mass = wq * cell**3
                exp_n += n * mass
                # continue the emitted tokens with the target model up to length K+1
                for tail in product(range(V), repeat=K + 1 - len(out)):
                    seq, m = out, mass
                    for t in tail:
                        m *= P[seq][t]
                        seq = seq + (t,)
                    law[seq] += m
        for s in law:
            want = P[()][s[0]] * P[s[:1]][s[1]] * P[s[:2]][s[2]]
            assert law[s] == want, (s, law[s], want)
        # E[n] = alpha_1 + E_{y1 accepted}[alpha_2], alpha = per-step overlap sum_v min(p_v, q_v)
        a1 = sum(min(a, b) for a, b in zip(P[()], Q[()]))
        a12 = sum(min(P[()][y], Q[()][y]) * sum(min(a, b) for a, b in zip(P[(y,)], Q[(y,)])) for y in range(V))
        assert exp_n == a1 + a12


def test_chained_law_matches_target_autoregression_exact():
    """Algorithm 2 with K=2: the emitted tokens, continued from the target model, follow the
    target's autoregressive law exactly (brute force over all drafts and a (r1,r2,u) grid)."""
    # V=2, entries in {1/4,1/2,3/4}: ratios below one are 1/3, 1/2, 2/3; CDFs in quarters -> G=12
    _chained_law_check(2, 12, [frac_array(["1/2", "1/2"]), frac_array(["1/4", "3/4"]), frac_array(["3/4", "1/4"])], 3, 5)
    # V=3, permutations of (1/4,1/4,1/2): ratio 1/2; residual CDFs in halves; p CDFs in quarters -> G=4
    perms = [frac_array(v) for v in (("1/4", "1/4", "1/2"), ("1/4", "1/2", "1/4"), ("1/2", "1/4", "1/4"))]
    _chained_law_check(3, 4, perms, 6, 6)


def test_ragged_length_equals_truncated_problem():
    """A row with cand_len = L inside a K-padded batch behaves as the K = L problem (Section 3.1)."""
    rng = np.random.default_rng(11)
    V, K = 9, 5
    t = rng.normal(size=(3, K + 1, V)).astype(np.float32)
    d = rng.normal(size=(3, K, V)).astype(np.float32)
    y = rng.integers(0, V, size=(3, K)).astype(np.int32)
    u = rng.random((3, K + 1)).astype(np.float32)
    lens = np.array([0, 2, 5], np.int32)
    full = orc.verify_correct(t, d, y, lens, u, 1.3)
    for b, L in enumerate(lens):
        ub = np.concatenate([u[b, :L], u[b, K:]])[None]
        one = orc.verify_correct(t[b:b + 1, :L + 1], d[b:b + 1, :L], y[b:b + 1, :L], None, ub, 1.3)
        assert one["n_accepted"][0] == full["n_accepted"][b]
        assert one["next_token"][0] == full["next_token"][b]


# ----------------------------------------------------------------------------- logits path
def test_softmax_and_lse_against_scipy():
    rng = np.random.default_rng(0)
    for T in (0.3, 0.7, 1.0, 2.5):
        z = rng.normal(scale=4.0, size=(5, 1000))
        Tf = float(np.float32(T))
        np.testing.assert_allclose(orc.softmax_T(z, T), scipy.special.softmax(z / Tf, axis=-1), rtol=1e-13)
        np.testing.assert_allclose(orc.log_sum_exp_T(z, T), scipy.special.logsumexp(z / Tf, axis=-1), rtol=1e-13)
    big = np.array([[1e4, 1e4 - 1.0, -1e4]])
    np.testing.assert_allclose(orc.softmax_T(big, 1.0)[0, :2], [1 / (1 + np.e**-1), np.e**-1 / (1 + np.e**-1)], rtol=1e-13)


def test_bf16_widening_is_exact():
    bits = np.arange(0, 1 << 16, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = orc.bf16_bits_to_f64(bits)
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite], ref[finite]) and np.array_equal(np.isnan(got), np.isnan(ref))


def test_inverse_cdf_is_upper_bound_search():
    rng = np.random.default_rng(3)
    for _ in range(200):
        V = int(rng.integers(1, 40))
        w = rng.random(V) * (rng.random(V) > 0.4)
        if w.sum() == 0:
            w[rng.integers(V)] = 1.0
        u = rng.random()
        c = np.cumsum(w)
        assert orc.inverse_cdf(w, u) == int(np.searchsorted(c, u * c[-1], side="right"))
    assert orc.inverse_cdf(np.array([0.0, 0.0, 2.0, 0.0]), 0.0) == 2     # zero-weight tokens never chosen
    assert orc.inverse_cdf(np.array([1.0, 0.0, 0.0]), 0.999999) == 0


def test_verify_correct_from_logits_matches_probability_form():
    """The logits entry point = scipy softmax followed by the probability-level algorithm."""
    rng = np.random.default_rng(21)
    B, K, V = 6, 4, 50
    t = rng.normal(scale=3, size=(B, K + 1, V)).astype(np.float32)
    d = (t[:, :K] + rng.normal(scale=1.0, size=(B, K, V))).astype(np.float32)
    y = rng.integers(0, V, size=(B, K)).astype(np.int32)
    u = rng.random((B, K + 1)).astype(np.float32)
    lens = rng.integers(0, K + 1, size=B).astype(np.int32)
    T = 0.8
    out = orc.verify_correct(t, d, y, lens, u, T)
    Tf = float(np.float32(T))
    for b in range(B):
        p = scipy.special.softmax(t[b].astype(np.float64) / Tf, axis=-1)
        q = scipy.special.softmax(d[b].astype(np.float64) / Tf, axis=-1)
        n, nxt, ratios, W = orc.verify_from_probs(p, q, y[b], int(lens[b]), u[b, :K].astype(np.float64), float(u[b, K]))
        assert (n, nxt) == (out["n_accepted"][b], out["next_token"][b])
        np.testing.assert_allclose(out["accept_ratio"][b, :lens[b]], np.minimum(1, ratios), rtol=1e-12)
        np.testing.assert_allclose(out["resid_mass"][b], W, rtol=1e-10)
        assert np.all(out["accept_ratio"][b, lens[b]:] == 0)


def test_mean_acceptance_equals_overlap_from_logits():
    """sum_y q(y) min(1, p(y)/q(y)) = sum_v min(p_v, q_v), using the oracle's ratios on every y."""
    rng = np.random.default_rng(8)
    V = 64
    t = rng.normal(scale=3, size=(1, 2, V)).astype(np.float32)
    d = rng.normal(scale=3, size=(1, 1, V)).astype(np.float32)
    p = scipy.special.softmax(t[0, 0].astype(np.float64))
    q = scipy.special.softmax(d[0, 0].astype(np.float64))
    acc = 0.0
    for y in range(V):
        o = orc.verify_correct(t, d, np.array([[y]], np.int32), None, np.zeros((1, 2), np.float32), 1.0)
        acc += q[y] * o["accept_ratio"][0, 0]
    np.testing.assert_allclose(acc, np.minimum(p, q).sum(), rtol=1e-12)


def test_special_cases():
    rng = np.random.default_rng(2)
    B, K, V = 4, 6, 37
    d = rng.normal(scale=3, size=(B, K, V)).astype(np.float32)
    t = np.concatenate([d, rng.normal(size=(B, 1, V)).astype(np.float32)], axis=1)
    y = rng.integers(0, V, size=(B, K)).astype(np.int32)
    u = rng.random((B, K + 1)).astype(np.float32)
    # p == q: every candidate is accepted (Appendix B discussion) and y' ~ p_{K+1}
    o = orc.verify_correct(t, d, y, None, u, 1.0)
    assert np.all(o["n_accepted"] == K)
    for b in range(B):
        pK = scipy.special.softmax(t[b, K].astype(np.float64))
        assert o["next_token"][b] == int(np.searchsorted(np.cumsum(pK), u[b, K] * np.cumsum(pK)[-1], side="right"))
    # very high temperature: both models uniform -> ratio 1 -> all accepted
    t2 = rng.normal(size=(B, K + 1, V)).astype(np.float32)
    assert np.all(orc.verify_correct(t2, d, y, None, u, 1e30)["n_accepted"] == K)
    # target essentially one-hot on the drafted token: accepted with ratio >= 1
    t3 = t2.copy()
    for b in range(B):
        t3[b, np.arange(K), y[b]] += 80.0
    o3 = orc.verify_correct(t3, d, y, None, u, 1.0)
    assert np.all(o3["n_accepted"] == K) and np.all(o3["accept_ratio"] == 1.0)
    # cand_len = 0: plain sampling from p_1
    o0 = orc.verify_correct(t2, d, y, np.zeros(B, np.int32), u, 1.0)
    assert np.all(o0["n_accepted"] == 0)
    for b in range(B):
        c = np.cumsum(scipy.special.softmax(t2[b, 0].astype(np.float64)))
        assert o0["next_token"][b] == int(np.searchsorted(c, u[b, K] * c[-1], side="right"))


def test_outputs_ignore_everything_after_first_rejection():
    """Tokens after the first rejection are discarded (Section 3.1): poison them and nothing changes."""
    rng = np.random.default_rng(4)
    B, K, V = 8, 6, 41
    d = rng.normal(scale=3, size=(B, K, V)).astype(np.float32)
    t = np.concatenate([d, d[:, :1]], axis=1) + rng.normal(scale=2.0, size=(B, K + 1, V)).astype(np.float32)
    y = rng.integers(0, V, size=(B, K)).astype(np.int32)
    u = rng.random((B, K + 1)).astype(np.float32)
    base = orc.verify_correct(t, d, y, None, u, 1.0)
    assert (base["n_accepted"] < K).any()
    t2, d2, y2, u2 = t.copy(), d.copy(), y.copy(), u.copy()
    for b in range(B):
        n = base["n_accepted"][b]
        t2[b, n + 1:] = rng.normal(scale=9, size=t2[b, n + 1:].shape)
        d2[b, n + 1:] = rng.normal(scale=9, size=d2[b, n + 1:].shape)
        y2[b, n + 1:] = (y2[b, n + 1:] + 1) % V
        u2[b, n + 1:K] = rng.random(K - n - 1) if n + 1 < K else u2[b, n + 1:K]
    again = orc.verify_correct(t2, d2, y2, None, u2, 1.0)
    assert np.array_equal(base["n_accepted"], again["n_accepted"])
    assert np.array_equal(base["next_token"], again["next_token"])


def test_monte_carlo_law_chi_square():
    """Secondary statistical check: 2e5 oracle draws at V=8 are compatible with p (chi-square, 7 dof)."""
    rng = np.random.default_rng(99)
    V, N = 8, 200_000
    t = rng.normal(scale=1.5, size=V)
    d = rng.normal(scale=1.5, size=V)
    p, q = scipy.special.softmax(t), scipy.special.softmax(d)
    ys = rng.choice(V, size=N, p=q)
    r, u = rng.random(N), rng.random(N)
    # vectorised use of the same primitives: accept where r < ratio, else inverse CDF of the residual
    ratio = p[ys] / q[ys]
    w = orc.residual(p, q)
    emitted = ys.copy()
    rej = np.nonzero(r >= ratio)[0]
    for idx in rej:
        emitted[idx] = orc.inverse_cdf(w, u[idx])
    counts = np.bincount(emitted, minlength=V)
    chi2 = ((counts - N * p) ** 2 / (N * p)).sum()
    assert chi2 < 29.9      # P(chi2_7 > 29.9) ~ 1e-4


# ----------------------------------------------------------------------------- stop rule
def test_stop_rule_closed_form_and_monotone():
    """Constant a in (0,1): first j with a^(j+1) < 1-h, i.e. j = floor(log(1-h)/log a) (strict)."""
    K = 40
    for a in (0.5, 0.8, 0.93, 0.99):
        for h in (0.1, 0.3, 0.5, 0.7, 0.9):
            probs = np.full((1, K), a, dtype=np.float32)
            a32, h32 = float(np.float32(a)), float(np.float32(h))
            x = np.log(1 - h32) / np.log(a32)
            if abs(x - round(x)) < 1e-6:
                continue
            want = int(np.floor(x))
            assert orc.stop_rule(probs, h)[0] == min(want, K)
    rng = np.random.default_rng(6)
    probs = rng.uniform(0.5, 1.0, size=(50, 16)).astype(np.float32)
    prev = np.zeros(50, np.int32)
    for h in np.linspace(-0.1, 1.1, 25):
        cur = orc.stop_rule(probs, h)
        assert np.all(cur >= prev)
        prev = cur
        # equivalent additive form: first j with sum -log a_i > -log(1-h)
        if 0 < h < 1:
            s = np.cumsum(-np.log(probs.astype(np.float64)), axis=1)
            hit = s > -np.log(1 - float(np.float32(h)))
            want = np.where(hit.any(1), hit.argmax(1), 16)
            near = np.abs(s - (-np.log(1 - float(np.float32(h))))).min(1) < 1e-9
            assert np.array_equal(cur[~near], want[~near])
    assert np.all(orc.stop_rule(probs, 1.0) == 16)            # h >= 1 never stops
    assert np.all(orc.stop_rule(probs, -0.01) == 0)           # h < 0 stops at once
    assert np.all(orc.stop_rule(np.ones((3, 5), np.float32), 0.0) == 5)
    lens = np.array([0, 2, 16], np.int32)
    out = orc.stop_rule(probs[:3], 0.999, lens)
    assert np.array_equal(out, lens)


def test_stop_step_iterated_equals_stop_rule():
    """Algorithm 1 applies the update one drafted token at a time; iterating it is the batched rule."""
    rng = np.random.default_rng(17)
    probs = rng.uniform(0.4, 1.0, size=(40, 12)).astype(np.float32)
    for h in (0.2, 0.5, 0.8):
        want = orc.stop_rule(probs, h)
        p_hat = np.ones(40)
        first = np.full(40, 12)
        for j in range(12):
            p_hat, stop = orc.stop_step(p_hat, probs[:, j], h)
            first = np.where((first == 12) & stop, j, first)
        assert np.array_equal(first, want)
    p, stop = orc.stop_step(np.array([1.0, 0.5]), np.array([0.5, 0.5], np.float32), 0.5)
    assert p.tolist() == [0.5, 0.25] and stop.tolist() == [False, True]      # strict: 1 - 0.5 > 0.5 is false


# ----------------------------------------------------------------------------- head
def _bf16(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_head_reduces_to_logistic_regression_and_identity():
    rng = np.random.default_rng(12)
    d = 32
    x = _bf16(rng.normal(size=(5, 3, d)))
    w = _bf16(rng.normal(scale=0.3, size=d))
    xf, wf = orc.bf16_bits_to_f64(x), orc.bf16_bits_to_f64(w)
    # D = 0: a linear layer followed by the logistic function
    got = orc.accept_head(x, [], w, 0.25)
    np.testing.assert_allclose(got, scipy.special.expit(xf @ wf + 0.25), rtol=1e-13)
    # zero blocks are the identity because SiLU(0) = 0
    Z = _bf16(np.zeros((d, d)))
    np.testing.assert_allclose(orc.accept_head(x, [(Z, None), (Z, _bf16(np.zeros(d)))], w, 0.25), got, rtol=1e-13)


def test_head_against_torch_float64_modules():
    """x <- x + SiLU(Wx+b) twice, then linear + sigmoid, evaluated by torch's own fp64 kernels."""
    rng = np.random.default_rng(13)
    d = 48
    x = _bf16(rng.normal(size=(7, d)))
    Ws = [_bf16(rng.normal(scale=0.2, size=(d, d))) for _ in range(2)]
    bs = [_bf16(rng.normal(scale=0.1, size=d)) for _ in range(2)]
    w = _bf16(rng.normal(scale=0.2, size=d))
    got = orc.accept_head(x, list(zip(Ws, bs)), w, -0.5)
    tx = torch.from_numpy(orc.bf16_bits_to_f64(x))
    for W, b in zip(Ws, bs):
        lin = torch.nn.functional.linear(tx, torch.from_numpy(orc.bf16_bits_to_f64(W)), torch.from_numpy(orc.bf16_bits_to_f64(b)))
        tx = tx + torch.nn.functional.silu(lin)
    want = torch.sigmoid(tx @ torch.from_numpy(orc.bf16_bits_to_f64(w)) - 0.5).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12)
    # a transposed weight would not survive this check
    assert not np.allclose(orc.accept_head(x, [(Ws[0].T.copy(), bs[0]), (Ws[1], bs[1])], w, -0.5), want, rtol=1e-3)


def test_top_k_filter_against_torch_topk_and_its_limits():
    """Appendix D.1's top-k sampling: the kept set is {v : z_v >= k-th largest} (library: torch.topk);
    k >= V changes nothing; k = 1 turns the stochastic algorithm into the greedy one of Section 4.1."""
    rng = np.random.default_rng(31)
    z = np.round(rng.normal(scale=2, size=(6, 200)) * 4) / 4           # quarter steps: ties at the threshold occur
    for k in (1, 5, 50, 199):
        kth = torch.topk(torch.from_numpy(z), k, dim=-1).values[:, -1:].numpy()
        want = np.where(z >= kth, z, -np.inf)
        got = orc.top_k_filter(z, k)
        assert np.array_equal(got, want)
        assert np.all((got > -np.inf).sum(-1) >= k)
    assert np.array_equal(orc.top_k_filter(z, 200), z) and np.array_equal(orc.top_k_filter(z, None), z)
    B, K, V = 10, 4, 64
    d = rng.normal(scale=2, size=(B, K, V)).astype(np.float32)
    t = np.concatenate([d, d[:, :1]], 1) + rng.normal(scale=1.5, size=(B, K + 1, V)).astype(np.float32)
    y = d.argmax(-1).astype(np.int32)
    u = rng.random((B, K + 1)).astype(np.float32)
    full = orc.verify_correct(t, d, y, None, u, 0.9)
    same = orc.verify_correct(t, d, y, None, u, 0.9, top_k=V)
    assert np.array_equal(full["n_accepted"], same["n_accepted"]) and np.array_equal(full["next_token"], same["next_token"])
    one = orc.verify_correct(t, d, y, None, u, 0.9, top_k=1)
    n_g, tok_g = orc.greedy_verify(t, d)
    assert np.array_equal(one["n_accepted"], n_g) and np.array_equal(one["next_token"], tok_g)
    # a drafted token outside the target's top-k is rejected with certainty; the draw stays inside it
    k = 5
    o = orc.verify_correct(t, d, y, None, u, 0.9, top_k=k)
    for b in range(B):
        n = o["n_accepted"][b]
        keep = np.argsort(-t[b, n].astype(np.float64), kind="stable")[:k]
        assert o["next_token"][b] in keep
        for i in range(K):
            if y[b, i] not in np.argsort(-t[b, i].astype(np.float64), kind="stable")[:k]:
                assert o["accept_ratio"][b, i] == 0.0


def test_greedy_case_is_the_low_temperature_limit():
    """Section 4.1: with greedy drafts the algorithm keeps candidates while they equal the target's
    argmax and emits the target's argmax at the first mismatch."""
    rng = np.random.default_rng(14)
    B, K, V = 12, 5, 23
    d = rng.normal(scale=2, size=(B, K, V)).astype(np.float32)
    t = np.concatenate([d, d[:, :1]], 1) + rng.normal(scale=1.2, size=(B, K + 1, V)).astype(np.float32)
    y = d.argmax(-1).astype(np.int32)
    u = rng.random((B, K + 1)).astype(np.float32)
    n_g, tok_g = orc.greedy_verify(t, d)
    cold = orc.verify_correct(t, d, y, None, u, 1e-3)
    assert np.array_equal(cold["n_accepted"], n_g) and np.array_equal(cold["next_token"], tok_g)


def test_greedy_ragged_lengths_equal_the_truncated_problem():
    """Section 4.1 on a ragged batch: a row of candidate length L is the K = L problem of its first
    L positions; rows of the target beyond position L are never looked at (they are poisoned with NaN
    here and must not change anything) and report -1 in target_argmax.  The expected values come from
    torch.argmax row by row, not from the function under test."""
    rng = np.random.default_rng(21)
    B, K, V = 9, 6, 17
    t = rng.normal(scale=2, size=(B, K + 1, V)).astype(np.float32)
    am_full = torch.from_numpy(t).double().argmax(-1).numpy()
    lens = np.array([0, 1, 2, 3, 4, 5, 6, 3, 6], np.int32)
    y = am_full[:, :K].astype(np.int32).copy()                 # all candidates match ...
    y[4, 2] = (y[4, 2] + 1) % V                                # ... except row 4 at position 2 (< L = 4)
    y[7, 3] = (y[7, 3] + 1) % V                                # row 7: mismatch at position 3 = L: not a candidate
    y[8, 0] = (y[8, 0] + 1) % V                                # row 8: first position mismatches
    tp, yp = t.copy(), y.copy()
    for b in range(B):
        tp[b, lens[b] + 1:] = np.nan
        yp[b, lens[b]:] = -7
    n, tok, am = orc.greedy_verify_tokens(tp, yp, lens)
    assert n.tolist() == [0, 1, 2, 3, 2, 5, 6, 3, 0]
    for b in range(B):
        assert tok[b] == am_full[b, n[b]]
        assert np.array_equal(am[b, :lens[b] + 1], am_full[b, :lens[b] + 1]) and np.all(am[b, lens[b] + 1:] == -1)
        # the truncated problem: K = L, no cand_len argument
        L = int(lens[b])
        if L >= 1:
            n1, tok1, _ = orc.greedy_verify_tokens(t[b:b + 1, :L + 1], y[b:b + 1, :L], None)
            assert (n1[0], tok1[0]) == (n[b], tok[b])
    # ties resolve to the lowest index
    tie = np.zeros((1, 2, 5), np.float32)
    tie[0, 0, [1, 3]] = 2.0
    n, tok, am = orc.greedy_verify_tokens(tie, np.array([[3]], np.int32), np.array([1], np.int32))
    assert (n[0], tok[0], am[0].tolist()) == (0, 1, [1, 0])


def test_drafted_token_with_zero_probability_under_both_models_is_rejected():
    """p(y) = q(y) = 0 (the logit of y is -inf in both rows): the ratio of the accept test is read as
    0, a certain rejection, as for any p(y) = 0; y' then comes from the residual, which gives y no
    weight.  Expected values from scipy's softmax and the probability-level core."""
    rng = np.random.default_rng(8)
    K, V = 3, 11
    d = rng.normal(scale=2, size=(1, K, V)).astype(np.float32)
    t = np.concatenate([d, d[:, :1]], 1) + rng.normal(size=(1, K + 1, V)).astype(np.float32)
    y = np.array([[2, 5, 7]], np.int32)
    t[0, 1, 5] = d[0, 1, 5] = -np.inf
    t[0, 0] = d[0, 0]                                          # position 0: p = q, accepted for any r < 1
    u = np.array([[0.999, 0.0, 0.5, 0.3]], np.float32)         # r_1 = 0 would accept any positive ratio
    o = orc.verify_correct(t, d, y, None, u, 1.0)
    assert o["n_accepted"][0] == 1 and o["accept_ratio"][0, 1] == 0.0 and o["p_y"][0, 1] == 0.0
    p = scipy.special.softmax(t[0].astype(np.float64), axis=-1)
    q = scipy.special.softmax(d[0].astype(np.float64), axis=-1)
    n, tok, ratios, W = orc.verify_from_probs(p, q, y[0], K, u[0, :K].astype(np.float64), float(u[0, K]))
    assert (n, tok) == (1, o["next_token"][0]) and ratios[1] == 0 and tok != 5
    # q(y) = 0 < p(y): always accepted
    t2, d2 = t.copy(), d.copy()
    t2[0, 1, 5] = 0.0
    o2 = orc.verify_correct(t2, d2, y, None, np.array([[0.999, 0.999, 0.999, 0.3]], np.float32), 1.0)
    assert o2["accept_ratio"][0, 1] == 1.0 and o2["n_accepted"][0] >= 2


# ----------------------------------------------------------------------------- planted mistakes
def test_pins_catch_planted_mistakes(monkeypatch):
    """Plant typical slips in the oracle (on the CPU) and check the exact-law pin notices."""
    p, q = frac_array(["1/10", "1/5", "3/10", "2/5"]), frac_array(["2/5", "3/10", "1/5", "1/10"])

    def law_ok():
        law = _emitted_law_one_step(p, q, 60)
        return all(law[x] == p[x] for x in range(4))

    assert law_ok()
    with monkeypatch.context() as m:          # residual with the sign flipped
        m.setattr(orc, "residual", lambda a, b: np.where(b - a > 0, b - a, (b - a) * 0))
        assert not law_ok()
    with monkeypatch.context() as m:          # ratio transposed
        m.setattr(orc, "accept_ratio", lambda a, b: b / a)
        assert not law_ok()
    with monkeypatch.context() as m:          # residual not clipped (dropped positive part)
        m.setattr(orc, "residual", lambda a, b: abs(a - b))
        assert not law_ok()
    with monkeypatch.context() as m:          # off-by-one in the CDF search
        real = orc.inverse_cdf
        m.setattr(orc, "inverse_cdf", lambda w, u: min(real(w, u) + 1, len(w) - 1))
        assert not law_ok()


def test_sample_law_on_a_dyadic_distribution():
    """Algorithm 1's draw y ~ q: with q = (1/8, 1/2, 1/4, 1/8) and u swept over the midpoints of a
    64-cell grid, every CDF breakpoint is a grid line, so the counts per token are exactly 64 q."""
    q = np.array([1 / 8, 1 / 2, 1 / 4, 1 / 8])
    u = (np.arange(64) + 0.5) / 64
    logits = np.tile(np.log(q) * 0.7 + 3.0, (64, 1))          # temperature and shift must cancel
    tok = orc.sample(logits, u, 0.7)
    assert np.bincount(tok, minlength=4).tolist() == [8, 32, 16, 8]
    assert np.all(np.diff(tok) >= 0)                           # vocabulary order
    # top-2 keeps tokens 1 and 2 with probabilities 2/3, 1/3 -> 96 cells: 64, 32
    u3 = (np.arange(96) + 0.5) / 96
    tok2 = orc.sample(np.tile(np.log(q), (96, 1)), u3, 1.0, top_k=2)
    assert np.bincount(tok2, minlength=4).tolist() == [0, 64, 32, 0]
