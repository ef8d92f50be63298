"""Helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same seeded
inputs and classify every row as exact, boundary-valid or wrong.

Boundary rule: discrete outputs must be identical, except where a uniform lies within 1e-6 of
the accept-ratio it is tested against or of an edge of the chosen token's CDF interval; such
rows are counted and reported, anything else fails.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import specdec_oracle as orc
from paper_2405_19715_b200 import specdec

BOUNDARY = 1e-6
PROB_RTOL = {"f32": 1e-5, "bf16": 2e-2}     # relative tolerances on probabilities by logit dtype


to_torch = specdec.from_numpy


def run_gpu_verify(ctx, inp, flags=0, want_stats=True):
    t, d = to_torch(inp["target_logits"]), to_torch(inp["draft_logits"])
    B, K1, V = t.shape
    K = K1 - 1
    y = to_torch(np.ascontiguousarray(inp["cand_tokens"], dtype=np.int32))
    L = None if inp.get("cand_len") is None else to_torch(np.ascontiguousarray(inp["cand_len"], dtype=np.int32))
    u = to_torch(np.ascontiguousarray(inp["uniforms"], dtype=np.float32))
    ratio = torch.full((B, K), -5.0, dtype=torch.float32, device="cuda") if want_stats else None
    stats = torch.full((B, K + 1, 4), -5.0, dtype=torch.float32, device="cuda") if want_stats else None
    mass = torch.full((B,), -5.0, dtype=torch.float32, device="cuda") if want_stats else None
    n, nxt = specdec.specdec_verify_correct(ctx, t, d, y, L, u, float(inp["temperature"]), accept_ratio=ratio,
                                            row_stats=stats, resid_mass=mass, flags=flags)
    torch.cuda.synchronize()
    out = dict(n_accepted=n.cpu().numpy(), next_token=nxt.cpu().numpy())
    if want_stats:
        out.update(accept_ratio=ratio.cpu().numpy(), row_stats=stats.cpu().numpy(), resid_mass=mass.cpu().numpy())
    return out


def _cdf_interval(w, g):
    c = np.cumsum(w)
    tot = c[-1]
    lo = (c[g - 1] if g > 0 else 0.0) / tot
    return lo, c[g] / tot, w[g]


def oracle_rows(inp, rows=None, top_k=None):
    """The oracle's outputs for `rows` (default all) of a problem: computed once and handed to
    classify_rows when several kernels are compared on the same inputs."""
    B, K1, _ = inp["target_logits"].shape
    rows = np.arange(B) if rows is None else np.array(list(rows))
    lens = np.full(B, K1 - 1, np.int32) if inp.get("cand_len") is None else np.asarray(inp["cand_len"])
    return orc.verify_correct(inp["target_logits"][rows], inp["draft_logits"][rows], inp["cand_tokens"][rows], lens[rows],
                              inp["uniforms"][rows], inp["temperature"], top_k=top_k)


def classify_rows(inp, gpu, rows=None, dtype="bf16", check_probs=True, top_k=None, oracle_out=None):
    """Compare GPU outputs with the oracle on `rows` (default all).  Returns a report dict and
    raises AssertionError on any row that is neither exact nor boundary-valid.  `mass_floor_rows`
    counts the rows whose residual mass agrees only through the absolute part of its tolerance."""
    tl, dl = inp["target_logits"], inp["draft_logits"]
    B, K1, V = tl.shape
    K = K1 - 1
    rows = list(range(B)) if rows is None else list(rows)
    T = inp["temperature"]
    lens = np.full(B, K, np.int32) if inp.get("cand_len") is None else np.asarray(inp["cand_len"])
    o = oracle_out if oracle_out is not None else oracle_rows(inp, rows, top_k)
    assert len(o["n_accepted"]) == len(rows)
    rep = dict(rows=len(rows), exact=0, boundary_n=0, boundary_token=0, max_ratio_rel=0.0, max_lse_abs=0.0,
               max_prob_rel=0.0, max_mass_rel=0.0, mass_floor_rows=0)
    rtol = PROB_RTOL[dtype]
    for k, b in enumerate(rows):
        L = int(lens[b])
        gn, gt = int(gpu["n_accepted"][b]), int(gpu["next_token"][b])
        on, ot = int(o["n_accepted"][k]), int(o["next_token"][k])
        r = inp["uniforms"][b].astype(np.float64)
        u = float(r[K])
        ratios = o["accept_ratio"][k]                      # min(1, p/q)
        assert 0 <= gn <= L, f"row {b}: n_accepted {gn} outside [0,{L}]"
        assert 0 <= gt < V, f"row {b}: next_token {gt} outside [0,{V})"
        n_boundary = False
        if gn != on:
            # every decision the GPU took that differs from the oracle's must sit on a boundary
            m = min(gn, on)
            assert abs(r[m] - ratios[m]) < BOUNDARY, f"row {b}: n {gn} vs oracle {on}, r-ratio={r[m]-ratios[m]:.3e}"
            for i in range(m + 1, gn):                     # GPU went on accepting: those must be accepts
                assert r[i] < ratios[i] + BOUNDARY, f"row {b}: position {i} accepted against the oracle"
            if gn < L and gn > m:
                assert r[gn] >= ratios[gn] - BOUNDARY, f"row {b}: position {gn} rejected against the oracle"
            n_boundary = True
            w = orc.sampling_weights(tl[b, gn], dl[b, gn] if gn < L else None, T, top_k)
            ot = orc.inverse_cdf(w, u)                     # the oracle's draw at the GPU's n
        if gt != ot:
            w = orc.sampling_weights(tl[b, gn], dl[b, gn] if gn < L else None, T, top_k)
            lo, hi, wg = _cdf_interval(w, gt)
            assert wg > 0 and lo - BOUNDARY <= u <= hi + BOUNDARY, \
                f"row {b}: token {gt} vs oracle {ot}: u={u!r} interval=({lo!r},{hi!r}) w={wg!r}"
            rep["boundary_token"] += 1
        elif n_boundary:
            rep["boundary_n"] += 1
        else:
            rep["exact"] += 1
        if not check_probs and "accept_ratio" in gpu:       # entry points without row_stats: ratios and mass only
            for i in range(L):
                rel = abs(gpu["accept_ratio"][b, i] - ratios[i]) / max(ratios[i], 1e-30)
                rep["max_ratio_rel"] = max(rep["max_ratio_rel"], rel if ratios[i] > 0 else abs(gpu["accept_ratio"][b, i]))
                assert (rel <= rtol) if ratios[i] > 0 else gpu["accept_ratio"][b, i] == 0, \
                    f"row {b} pos {i}: accept ratio {gpu['accept_ratio'][b, i]!r} vs {ratios[i]!r}"
            if gn == on and "resid_mass" in gpu:
                assert abs(gpu["resid_mass"][b] - o["resid_mass"][k]) <= rtol * o["resid_mass"][k] + 1e-6
                rep["mass_floor_rows"] += int(abs(gpu["resid_mass"][b] - o["resid_mass"][k]) > rtol * o["resid_mass"][k])
        if check_probs and "accept_ratio" in gpu:
            ga, st = gpu["accept_ratio"][b], gpu["row_stats"][b]
            for i in range(L):
                rel = abs(ga[i] - ratios[i]) / max(ratios[i], 1e-30)
                rep["max_ratio_rel"] = max(rep["max_ratio_rel"], rel)
                assert rel <= rtol, f"row {b} pos {i}: accept ratio {ga[i]!r} vs {ratios[i]!r}"
                for gv, ov in ((st[i, 2], o["p_y"][k, i]), (st[i, 3], o["q_y"][k, i])):
                    rel = abs(gv - ov) / max(ov, 1e-30)
                    if ov > 1e-30:
                        rep["max_prob_rel"] = max(rep["max_prob_rel"], rel)
                        assert rel <= rtol, f"row {b} pos {i}: prob {gv!r} vs {ov!r}"
                for gv, ov in ((st[i, 0], o["lse_p"][k, i]), (st[i, 1], o["lse_q"][k, i])):
                    rep["max_lse_abs"] = max(rep["max_lse_abs"], abs(gv - ov))
                    assert abs(gv - ov) <= 1e-5 * max(1.0, abs(ov)), f"row {b} pos {i}: lse {gv!r} vs {ov!r}"
            assert np.all(ga[L:] == 0), f"row {b}: accept_ratio beyond cand_len not zero"
            assert np.all(st[L + 1:] == 0) and np.all(st[L, 1:] == 0), f"row {b}: row_stats beyond cand_len not zero"
            if gn == on:
                gm, om = gpu["resid_mass"][b], o["resid_mass"][k]
                rel = abs(gm - om) / max(om, 1e-30)
                rep["max_mass_rel"] = max(rep["max_mass_rel"], rel)
                # W = sum (p-q)_+ cancels: fp32 probabilities carry ~1e-7 each, so the bound is absolute
                assert abs(gm - om) <= rtol * om + 1e-6, f"row {b}: residual mass {gm!r} vs {om!r}"
                rep["mass_floor_rows"] += int(abs(gm - om) > rtol * om)
                if gn == L:
                    assert abs(st[L, 0] - o["lse_p"][k, L]) <= 1e-5 * max(1.0, abs(o["lse_p"][k, L])), \
                        f"row {b}: bonus lse {st[L, 0]!r} vs {o['lse_p'][k, L]!r} (L={L}, stats={st.tolist()})"
    return rep


def classify_stop(accept_prob, h, gpu_pos, cand_len=None):
    """Stop-rule parity: exact, or boundary-valid when |1 - prod - h| < 1e-6 at a disputed position."""
    a = np.asarray(accept_prob, dtype=np.float32)
    B, K = a.shape
    o = orc.stop_rule(a, h, cand_len)
    lens = np.full(B, K) if cand_len is None else np.asarray(cand_len)
    hf = float(np.float32(h))
    rep = dict(rows=B, exact=0, boundary=0)
    for b in range(B):
        if gpu_pos[b] == o[b]:
            rep["exact"] += 1
            continue
        c = np.cumprod(a[b].astype(np.float64))
        lo, hi = sorted((int(gpu_pos[b]), int(o[b])))
        assert 0 <= lo and hi <= lens[b], f"row {b}: stop_pos {gpu_pos[b]} outside [0,{lens[b]}]"
        for j in range(lo, min(hi + 1, int(lens[b]))):
            if j == hi and hi == lens[b]:
                break
            if (j < hi):
                assert abs(1.0 - c[j] - hf) < BOUNDARY, f"row {b}: stop_pos {gpu_pos[b]} vs oracle {o[b]}"
        rep["boundary"] += 1
    return rep
