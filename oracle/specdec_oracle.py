"""CPU oracle for the SpecDec++ verify/correct step, acceptance head and stop rule.

THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  Only the tests, the smoke check
and the benchmark's CPU-baseline leg may import it.  It shares no code with the CUDA
library and never calls it.  Everything is plain numpy in float64 (or, for the exact
pins, numpy object arrays holding ``fractions.Fraction``); there is no blocking,
fusion or reordering beyond what the paper's algorithm states.

What it follows (arXiv 2405.19715):
  * Appendix C, "Rejection Sampling" paragraph: accept x~q with probability
    min(1, p(x)/q(x)), otherwise draw from Norm[(p-q)_+].
  * Algorithm 2 (and the lower half of Algorithm 1): uniforms r_i, the count
    n = min({i-1 : r_i >= p_i(y_i)/q_i(y_i)} U {K}), the residual draw when n < K and
    the draw from p_{K+1} when n = K.
  * Section 4.3 / Eq. 3: predicted acceptance = sigmoid(f_theta(e_i)); stop when
    1 - prod_i sigmoid(f_theta(e_i)) > h (chain rule, strict inequality).
  * Section 5.1: f_theta is a (D+1)-layer ResNet with SiLU activations.
  * Appendix D.1: sampling temperature T (the paper runs T = 1).

Readings taken where the paper is silent (each is also listed in the design notes):
  * positions are 0-based here; row ``L`` of the target tensor is the paper's
    p_{K+1} for a row whose candidate length is L (ragged batches);
  * equality r_i == ratio rejects (the paper writes ">=");
  * y' is drawn by inverse CDF in vocabulary order from one extra uniform u:
    the smallest j with sum_{v<=j} w_v > u * sum_v w_v (strict, so zero-weight
    tokens are never chosen);
  * a residual with zero total mass (p == q to rounding) falls back to p_n;
  * the head block is x <- x + SiLU(W x + b), D blocks, then a linear d -> 1.

Parity pins: every function below is pinned by tests/test_oracle_pins.py against
exact-rational brute force, closed forms, invariants or an independent library
routine, except ``accept_head`` evaluated on *trained* weights, for which no
published values exist: parity unpinned for trained-weight outputs (its
arithmetic is pinned through the D=0 logistic case, the zero-weight identity and
an independent library evaluation on random weights).
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "bf16_bits_to_f64", "logits_to_f64", "softmax_T", "log_sum_exp_T",
    "accept_ratio", "first_rejection", "residual", "inverse_cdf",
    "verify_from_probs", "verify_correct", "sampling_weights", "top_k_filter",
    "silu", "sigmoid", "accept_head", "stop_rule", "greedy_verify", "greedy_verify_tokens", "stop_step",
]


# --------------------------------------------------------------------------- storage
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64.

    bfloat16 is the upper half of an IEEE-754 binary32, so the value is the binary32
    whose low 16 mantissa bits are zero; binary32 -> binary64 is exact.
    """
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    with np.errstate(invalid="ignore"):      # signalling-NaN patterns widen to quiet NaN
        return b.view(np.float32).astype(np.float64)


def logits_to_f64(x: np.ndarray) -> np.ndarray:
    """Stored logits (float32, float64, or uint16 = bfloat16 bits) as float64, exactly."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return bf16_bits_to_f64(x)
    return x.astype(np.float64)


# --------------------------------------------------------------------------- softmax
def _temperature(T) -> float:
    # The library receives T as a C float; the oracle uses exactly that value.
    t = float(np.float32(T))
    if not (t > 0.0) or not np.isfinite(t):
        raise ValueError("temperature must be a positive finite float")
    return t


def softmax_T(z: np.ndarray, T) -> np.ndarray:
    """p = softmax(z / T) over the last axis, max-subtracted (Appendix D.1 temperature)."""
    x = np.asarray(z, dtype=np.float64) / _temperature(T)
    x = x - np.max(x, axis=-1, keepdims=True)
    e = np.exp(x)
    return e / np.sum(e, axis=-1, keepdims=True)


def log_sum_exp_T(z: np.ndarray, T) -> np.ndarray:
    """log sum_v exp(z_v / T) over the last axis."""
    x = np.asarray(z, dtype=np.float64) / _temperature(T)
    m = np.max(x, axis=-1, keepdims=True)
    return (m + np.log(np.sum(np.exp(x - m), axis=-1, keepdims=True)))[..., 0]


def top_k_filter(z: np.ndarray, k) -> np.ndarray:
    """Top-k sampling filter (Appendix D.1: the paper samples with k = 50): logits below the k-th
    largest of the row become -inf, so their probability is zero; ties with the k-th largest are
    kept.  k = None or k >= V leaves the row unchanged."""
    z = np.asarray(z, dtype=np.float64)
    if k is None or k >= z.shape[-1]:
        return z
    kth = np.sort(z, axis=-1)[..., -int(k)][..., None]
    return np.where(z >= kth, z, -np.inf)


# --------------------------------------------------------------------------- one rejection step
def accept_ratio(p_y, q_y):
    """p(y)/q(y) of the drafted token (Appendix C; Algorithm 2's acceptance test).

    The caller draws y from q, so q(y) > 0 whenever the ratio matters; q(y) == 0
    gives +inf (accept) if p(y) > 0 and 0 (reject) otherwise.
    """
    if q_y == 0:
        return float("inf") if p_y > 0 else 0
    return p_y / q_y


def first_rejection(ratios, r, L: int) -> int:
    """n = min({i : r_i >= ratio_i, i < L} U {L}) with 0-based i (Algorithm 2)."""
    for i in range(L):
        if r[i] >= ratios[i]:
            return i
    return L


def residual(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    """(p - q)_+ elementwise, un-normalised (Appendix C)."""
    d = p - q
    return np.where(d > 0, d, d * 0)


def inverse_cdf(w: np.ndarray, u) -> int:
    """Smallest j with sum_{v<=j} w_v > u * sum_v w_v; plain left-to-right sums.

    Draws from Norm[w] when u ~ Unif[0,1): token j owns the interval
    [F_{j-1}, F_j) of the normalised CDF.
    """
    c = np.cumsum(w)            # sequential, vocabulary order
    total = c[-1]
    thr = u * total
    hit = np.nonzero(c > thr)[0]
    if hit.size == 0:           # only reachable through rounding (or u >= 1)
        pos = np.nonzero(w > 0)[0]
        return int(pos[-1]) if pos.size else int(len(w) - 1)
    return int(hit[0])


def verify_from_probs(p, q, y, L: int, r, u):
    """One row of Algorithm 2 given the distributions themselves.

    p: [>=L+1, V] target distributions, q: [>=L, V] draft distributions (float64 or
    Fraction objects), y: drafted tokens, r: uniforms for the accept tests, u: the
    uniform for y'.  Returns (n, y_next, ratios[0:L], W) where W is the residual mass
    at n (1 for the bonus draw).
    """
    ratios = [accept_ratio(p[i][y[i]], q[i][y[i]]) for i in range(L)]
    n = first_rejection(ratios, r, L)
    if n < L:
        w = residual(p[n], q[n])
        W = np.cumsum(w)[-1]
        if not (W > 1e-30):     # p == q up to rounding: nothing to renormalise
            w, W = p[n], np.cumsum(p[n])[-1]
    else:
        w = p[L]
        W = np.cumsum(w)[-1]
    return n, inverse_cdf(w, u), ratios, W


# --------------------------------------------------------------------------- batched, from logits
def sampling_weights(target_row, draft_row, T, top_k=None):
    """Un-normalised weights y' is drawn from at one position: (p - q)_+ when a draft
    row is given (rejection), p itself when ``draft_row`` is None (bonus).  With ``top_k`` both
    distributions are the top-k filtered ones."""
    p = softmax_T(top_k_filter(logits_to_f64(target_row), top_k), T)
    if draft_row is None:
        return p
    w = residual(p, softmax_T(top_k_filter(logits_to_f64(draft_row), top_k), T))
    if not (np.cumsum(w)[-1] > 1e-30):
        return p
    return w


def verify_correct(target_logits, draft_logits, cand_tokens, cand_len, uniforms, T, top_k=None):
    """Batched verify + correct (Algorithm 2, lower half of Algorithm 1).

    target_logits [B,K+1,V], draft_logits [B,K,V] (float32 or uint16 bf16 bits),
    cand_tokens [B,K] int, cand_len [B] int or None (all K), uniforms [B,K+1] float32
    ([b,i<K] = r_i, [b,K] = u for y').  Positions at or beyond cand_len[b] (and target
    rows beyond cand_len[b]) are never touched.

    Returns a dict: n_accepted [B], next_token [B], accept_ratio [B,K] = min(1, p/q)
    (0 beyond cand_len), lse_p [B,K+1], lse_q [B,K], p_y, q_y [B,K], resid_mass [B].
    """
    target_logits = np.asarray(target_logits)
    draft_logits = np.asarray(draft_logits)
    B, K1, V = target_logits.shape
    K = K1 - 1
    T = _temperature(T)
    cand_tokens = np.asarray(cand_tokens).reshape(B, K)
    uniforms = np.asarray(uniforms, dtype=np.float32).astype(np.float64).reshape(B, K + 1)
    lens = np.full(B, K, dtype=np.int64) if cand_len is None else np.asarray(cand_len, dtype=np.int64)
    out = dict(
        n_accepted=np.zeros(B, np.int32), next_token=np.zeros(B, np.int32),
        accept_ratio=np.zeros((B, K)), lse_p=np.zeros((B, K + 1)), lse_q=np.zeros((B, K)),
        p_y=np.zeros((B, K)), q_y=np.zeros((B, K)), resid_mass=np.zeros(B),
    )
    for b in range(B):
        L = int(lens[b])
        if not (0 <= L <= K):
            raise ValueError(f"cand_len[{b}]={L} outside [0,{K}]")
        ratios = []
        for i in range(L):
            y = int(cand_tokens[b, i])
            if not (0 <= y < V):
                raise ValueError(f"cand_tokens[{b},{i}]={y} outside [0,{V})")
            t = top_k_filter(logits_to_f64(target_logits[b, i]), top_k)
            d = top_k_filter(logits_to_f64(draft_logits[b, i]), top_k)
            lp, lq = log_sum_exp_T(t, T), log_sum_exp_T(d, T)
            log_py, log_qy = t[y] / T - lp, d[y] / T - lq
            if log_py == -np.inf:                    # p_i(y_i) = 0 (filtered out): certain rejection
                ratio = 0.0
            elif log_qy == -np.inf:                  # q_i(y_i) = 0 < p_i(y_i)
                ratio = np.inf
            else:
                ratio = np.exp(log_py - log_qy)      # = p_i(y_i) / q_i(y_i)
            ratios.append(ratio)
            out["lse_p"][b, i], out["lse_q"][b, i] = lp, lq
            out["p_y"][b, i], out["q_y"][b, i] = np.exp(log_py), np.exp(log_qy)
            out["accept_ratio"][b, i] = min(1.0, ratio)
        n = first_rejection(ratios, uniforms[b, :K], L)
        if n < L:
            w = sampling_weights(target_logits[b, n], draft_logits[b, n], T, top_k)
            pn = softmax_T(top_k_filter(logits_to_f64(target_logits[b, n]), top_k), T)
            qn = softmax_T(top_k_filter(logits_to_f64(draft_logits[b, n]), top_k), T)
            out["resid_mass"][b] = np.cumsum(residual(pn, qn))[-1]
        else:
            out["lse_p"][b, L] = log_sum_exp_T(top_k_filter(logits_to_f64(target_logits[b, L]), top_k), T)
            w = sampling_weights(target_logits[b, L], None, T, top_k)
            out["resid_mass"][b] = 1.0
        out["n_accepted"][b] = n
        out["next_token"][b] = inverse_cdf(w, uniforms[b, K])
    return out


def sample(logits, uniforms, T, top_k=None):
    """Algorithm 1's drafting draw y ~ softmax(logits / T) for every row of logits [B, V] (also the
    K = 0 round of Algorithm 2 on the target's logits): inverse CDF in vocabulary order at
    uniforms[b], after the top-k filter of Appendix D.1 when top_k is given."""
    z = logits_to_f64(logits)
    u = np.asarray(uniforms, dtype=np.float64).reshape(-1)
    return np.array([inverse_cdf(sampling_weights(z[b], None, T, top_k), u[b]) for b in range(z.shape[0])],
                    dtype=np.int64)


def greedy_verify_tokens(target_logits, cand_tokens, cand_len=None):
    """Greedy special case (Section 4.1) with the drafted tokens given: a candidate is kept while
    it equals argmax p_i, the first mismatch is replaced by argmax p_i, and argmax p_L is appended
    when all L candidates match.  Ties resolve to the lowest index.  Returns (n_accepted,
    next_token, target_argmax [B,K+1] with -1 at rows the method does not look at)."""
    t = logits_to_f64(np.asarray(target_logits))
    B, K1, _ = t.shape
    y = np.asarray(cand_tokens).reshape(B, K1 - 1)
    lens = np.full(B, K1 - 1) if cand_len is None else np.asarray(cand_len)
    n_acc, nxt = np.zeros(B, np.int32), np.zeros(B, np.int32)
    am = np.full((B, K1), -1, np.int32)
    for b in range(B):
        L = int(lens[b])
        for i in range(L + 1):
            am[b, i] = int(np.argmax(t[b, i]))
        n = L
        for i in range(L):
            if int(y[b, i]) != am[b, i]:
                n = i
                break
        n_acc[b], nxt[b] = n, am[b, n]
    return n_acc, nxt, am


def greedy_verify(target_logits, draft_logits, cand_len=None):
    """Greedy special case (Section 4.1): the draft proposes argmax q_i; see greedy_verify_tokens."""
    d = logits_to_f64(np.asarray(draft_logits))
    n_acc, nxt, _ = greedy_verify_tokens(target_logits, d.argmax(-1), cand_len)
    return n_acc, nxt


# --------------------------------------------------------------------------- head + stop rule
def silu(x):
    """SiLU(x) = x * sigmoid(x)."""
    return x * sigmoid(x)


def sigmoid(x):
    """1 / (1 + exp(-x)), evaluated without overflow for either sign."""
    x = np.asarray(x, dtype=np.float64)
    e = np.exp(-np.abs(x))
    return np.where(x >= 0, 1.0 / (1.0 + e), e / (1.0 + e))


def accept_head(hidden, blocks, w_out, b_out):
    """sigmoid(f_theta(e)) of Eq. 3 with f_theta a (D+1)-layer ResNet (Section 5.1).

    hidden [..., d]; blocks = [(W_1, b_1), ..., (W_D, b_D)] with W_k [d, d] stored
    (out, in) and b_k [d] or None; w_out [d], b_out scalar.  Each block is
    x <- x + SiLU(W_k x + b_k); the last layer is w_out . x + b_out.  Inputs may be
    bf16 bit patterns; all arithmetic is float64 with no intermediate rounding.
    """
    x = logits_to_f64(hidden)
    for W, b in blocks:
        z = x @ logits_to_f64(W).T
        if b is not None:
            z = z + logits_to_f64(b)
        x = x + silu(z)
    return sigmoid(x @ logits_to_f64(w_out) + float(b_out))


def stop_rule(accept_prob, h, cand_len=None):
    """First 0-based j with 1 - prod_{i<=j} a_i > h (Section 4.3; Algorithm 1's loop).

    accept_prob [B,K] float32 values (used exactly, in float64).  Returns stop_pos [B]:
    j, or cand_len[b] (K when None) if the rule never fires within the row.
    """
    a = np.asarray(accept_prob, dtype=np.float32).astype(np.float64)
    B, K = a.shape
    h = float(np.float32(h))
    lens = np.full(B, K) if cand_len is None else np.asarray(cand_len)
    out = np.zeros(B, np.int32)
    for b in range(B):
        c, pos = 1.0, int(lens[b])
        for j in range(int(lens[b])):
            c = c * a[b, j]
            if 1.0 - c > h:
                pos = j
                break
        out[b] = pos
    return out


def stop_step(p_hat, accept_prob_step, h):
    """One trip of Algorithm 1's drafting loop for a batch: p_hat <- p_hat * sigmoid(f(e)) and the
    decision 1 - p_hat > h.  p_hat, accept_prob_step: [B] float32 values (used exactly, in float64).
    Returns (new p_hat [B] float64, stop [B] bool)."""
    p = np.asarray(p_hat, dtype=np.float64) * np.asarray(accept_prob_step, dtype=np.float32).astype(np.float64)
    return p, (1.0 - p) > float(np.float32(h))

