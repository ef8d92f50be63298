"""A float64 CPU model of the three local phases of vocabulary-sharded verify/correct, built from the
oracle's pinned pieces.  It stands in for the CUDA binding so that the exchange protocol
(`paper_2405_19715_b200.sharded`) can run on gloo ranks without a GPU; its own correctness is checked
by comparing the protocol's result with the oracle on the concatenated logits."""
import numpy as np
import torch

from oracle import specdec_oracle as orc


def _np(t):
    return None if t is None else t.numpy()


def specdec_shard_stats(ctx, target_shard, draft_shard, v_offset, V, cand_tokens, cand_len, temperature):
    t, d = orc.logits_to_f64(_np(target_shard)), orc.logits_to_f64(_np(draft_shard))
    B, K1, Vs = t.shape
    K = K1 - 1
    lens = np.full(B, K) if cand_len is None else _np(cand_len)
    rec = np.zeros((B, K1, 8))
    rec[:, :, 0] = rec[:, :, 2] = -np.inf
    for b in range(B):
        for i in range(lens[b] + 1):
            z = t[b, i] / temperature
            rec[b, i, 0], rec[b, i, 1] = z.max(), np.exp(z - z.max()).sum()
            if i < lens[b]:
                zq = d[b, i] / temperature
                rec[b, i, 2], rec[b, i, 3] = zq.max(), np.exp(zq - zq.max()).sum()
                y = int(cand_tokens[b, i]) - v_offset
                if 0 <= y < Vs:
                    rec[b, i, 4:7] = t[b, i, y], d[b, i, y], 1.0
    return torch.from_numpy(rec)


def _lse(stats_all, b, i, col):
    m = stats_all[:, b, i, col]
    s = stats_all[:, b, i, col + 1]
    top = m.max()
    return top + np.log((s * np.exp(m - top)).sum())


def _weights(t, d, b, n, L, T, lse_p, lse_q):
    p = np.exp(t[b, n] / T - lse_p)
    return p if n == L else np.maximum(p - np.exp(d[b, n] / T - lse_q), 0.0)


def specdec_shard_accept(ctx, target_shard, draft_shard, v_offset, V, stats_all, cand_len, uniforms, temperature,
                         accept_ratio=None):
    t, d = orc.logits_to_f64(_np(target_shard)), orc.logits_to_f64(_np(draft_shard))
    sa = stats_all.numpy()
    B, K1, _ = t.shape
    K = K1 - 1
    lens = np.full(B, K) if cand_len is None else _np(cand_len)
    u = uniforms.numpy().astype(np.float64)
    n_acc = np.zeros(B, np.int32)
    norm = np.zeros((B, 4))
    mass = np.zeros(B)
    for b in range(B):
        n = lens[b]
        for i in range(lens[b]):
            ty, dy = sa[:, b, i, 4].sum(), sa[:, b, i, 5].sum()
            ratio = np.exp((ty - dy) / temperature - _lse(sa, b, i, 0) + _lse(sa, b, i, 2))
            if u[b, i] >= ratio:
                n = i
                break
        n_acc[b] = n
        lp = _lse(sa, b, n, 0)
        lq = _lse(sa, b, n, 2) if n < lens[b] else lp
        norm[b] = lp, 0.0, lq, 0.0
        mass[b] = _weights(t, d, b, n, lens[b], temperature, lp, lq).sum()
    return torch.from_numpy(n_acc), torch.from_numpy(norm), torch.from_numpy(mass)


def specdec_shard_draw(ctx, target_shard, draft_shard, v_offset, V, stats_all, mass_all, rank, n_accepted, cand_len,
                       uniforms, row_norm, temperature, resid_mass=None):
    t, d = orc.logits_to_f64(_np(target_shard)), orc.logits_to_f64(_np(draft_shard))
    B, K1, _ = t.shape
    K = K1 - 1
    lens = np.full(B, K) if cand_len is None else _np(cand_len)
    ma, nr, u = mass_all.numpy(), row_norm.numpy(), uniforms.numpy().astype(np.float64)
    out = np.full(B, -1, np.int32)
    for b in range(B):
        thr = u[b, K] * ma[:, b].sum()
        cum = np.cumsum(ma[:, b])
        owner = int(np.argmax(cum > thr))
        if owner != rank:
            continue
        before = cum[owner] - ma[owner, b]
        n = int(n_accepted[b])
        w = _weights(t, d, b, n, lens[b], temperature, nr[b, 0], nr[b, 2])
        c = before + np.cumsum(w)
        hit = np.nonzero((c > thr) & (w > 0))[0]
        out[b] = v_offset + (int(hit[0]) if len(hit) else int(np.nonzero(w > 0)[0][-1]))
    return torch.from_numpy(out)
