"""Seeded synthetic inputs for the verify/correct, head and stop-rule entry points.

This module only *draws inputs*: normal logits, candidate tokens, uniforms, hidden
states and head weights, with the shapes and value distributions of the five
workloads below.  It contains none of the method's arithmetic (no softmax, no accept
test, no residual, no inverse CDF, no head forward, no stop rule), so both the CUDA
library's tests and the CPU oracle's tests can consume the same bytes.

All randomness comes from numpy's Philox counter-based generator keyed by
(seed, tensor id, batch row), so any row of any tensor can be regenerated alone and
the result does not depend on thread count.  bfloat16 tensors are returned as
``uint16`` bit patterns (round-to-nearest-even from float32).

Workloads (the vocabulary size 32000 is that of the llama-2 pair the paper decodes
with, candidate lengths up to 16 sit inside its 2..20 range, T = 1 is its sampling
temperature; the synthetic logits stand in for the Alpaca / HumanEval / GSM8K runs
of Section 5, whose prompts and weights are not available):

  cfg1  B=1   K=4   V=32000   fp32  draft N(0,3^2), target = draft + N(0,1),   T=1.0
  cfg2  B=8   K=8   V=32000   bf16  draft N(0,3^2), target = draft + N(0,.7^2), T=0.7
  cfg3  B=64  K=16  V=32000   bf16  ragged cand_len ~ U{1..16}, per-row noise
                                    sigma ~ U(0.3,2.0), T=1.0, padding poisoned
  cfg4  B=256 K=16  V=128256  bf16  draft N(0,4^2), target = draft + N(0,1), 10 % of
                                    rows get +12 on the drafted token's target logit
  cfg5  B=128 K=16  V=32000   bf16  logits as cfg2; hidden [B,K,4096] N(0,1) and a
                                    D=2 residual head with N(0,0.02^2) weights
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 240519715

_TENSOR_IDS = {"base": 1, "noise": 2, "gumbel": 3, "uniforms": 4, "cand_len": 5, "sigma": 6,
               "peaked": 7, "hidden": 8, "W": 9, "w_out": 10, "accept_prob": 11, "bonus_peak": 12}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    K: int
    V: int
    dtype: str                 # "f32" or "bf16": storage type of the logits
    sigma_d: float
    sigma_n: float             # noise std (ignored when sigma_n_range is set)
    T: float
    sigma_n_range: tuple | None = None   # per-row noise std ~ U(lo, hi)
    ragged: bool = False       # cand_len ~ U{1..K}; padding filled with a sentinel
    peaked_frac: float = 0.0   # fraction of rows whose drafted token gets +peak on target
    peak: float = 12.0
    d: int = 0                 # hidden width (0 = no head inputs)
    depth: int = 0             # number of residual blocks D
    h: float = 0.5
    seed: int = BASE_SEED

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS = {
    "cfg1": Workload("cfg1", B=1, K=4, V=32000, dtype="f32", sigma_d=3.0, sigma_n=1.0, T=1.0),
    "cfg2": Workload("cfg2", B=8, K=8, V=32000, dtype="bf16", sigma_d=3.0, sigma_n=0.7, T=0.7),
    "cfg3": Workload("cfg3", B=64, K=16, V=32000, dtype="bf16", sigma_d=3.0, sigma_n=1.0, T=1.0,
                     sigma_n_range=(0.3, 2.0), ragged=True),
    "cfg4": Workload("cfg4", B=256, K=16, V=128256, dtype="bf16", sigma_d=4.0, sigma_n=1.0, T=1.0,
                     peaked_frac=0.10),
    "cfg5": Workload("cfg5", B=128, K=16, V=32000, dtype="bf16", sigma_d=3.0, sigma_n=0.7, T=0.7,
                     d=4096, depth=2, h=0.5),
}

# bf16 pattern written into logits that must never be read (rows past cand_len).
SENTINEL_BF16 = np.uint16(0x7FC0)      # quiet NaN
SENTINEL_F32 = np.float32(np.nan)


def _rng(seed: int, tensor: str, row: int = 0) -> np.random.Generator:
    key = np.array([seed & 0xFFFFFFFFFFFFFFFF, (_TENSOR_IDS[tensor] << 40) | (row & 0xFFFFFFFFFF)],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest even (NaN kept quiet)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    b = x.view(np.uint32)
    rounded = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = SENTINEL_BF16
    return out


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(x) if dtype == "bf16" else np.array(x, dtype=np.float32, order="C", copy=True)


def _stored_as_f32(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return x


def uniforms_24bit(rng: np.random.Generator, shape) -> np.ndarray:
    """k / 2^24 with k uniform on [0, 2^24): exactly representable float32 in [0,1)."""
    k = rng.integers(0, 1 << 24, size=shape, dtype=np.int64)
    return (k.astype(np.float64) / float(1 << 24)).astype(np.float32)


def make_cand_len(wl: Workload) -> np.ndarray:
    if not wl.ragged:
        return np.full(wl.B, wl.K, dtype=np.int32)
    return _rng(wl.seed, "cand_len").integers(1, wl.K + 1, size=wl.B).astype(np.int32)


def _row_logits(wl: Workload, b: int, L: int, sigma_n: float, peaked: bool):
    """Logits, candidate tokens for batch row b.  Returns (target [K+1,V], draft [K,V], y [K])."""
    K, V = wl.K, wl.V
    base = _rng(wl.seed, "base", b).standard_normal((K + 1, V), dtype=np.float32) * np.float32(wl.sigma_d)
    draft = _store(base[:K], wl.dtype)
    # Candidate tokens y_i ~ softmax(draft_i / T), drawn with the Gumbel-max construction
    # on the *stored* draft logits (Section 3.1: y_i ~ q_i).
    g = _rng(wl.seed, "gumbel", b).gumbel(size=(K, V)).astype(np.float32)
    y = np.argmax(_stored_as_f32(draft, wl.dtype) / np.float32(wl.T) + g, axis=1).astype(np.int32)
    del g
    base += _rng(wl.seed, "noise", b).standard_normal((K + 1, V), dtype=np.float32) * np.float32(sigma_n)
    if peaked:
        base[np.arange(K), y] += np.float32(wl.peak)
        base[K, int(_rng(wl.seed, "bonus_peak", b).integers(0, V))] += np.float32(wl.peak)
    target = _store(base, wl.dtype)
    if L < K:   # poison everything the method must not read
        if wl.dtype == "bf16":
            target[L + 1:], draft[L:] = SENTINEL_BF16, SENTINEL_BF16
        else:
            target[L + 1:], draft[L:] = SENTINEL_F32, SENTINEL_F32
        y[L:] = -7
    return target, draft, y


def make_verify_inputs(wl: Workload, threads: int | None = None) -> dict:
    """All inputs of one verify/correct call for workload ``wl`` (numpy, host memory)."""
    B, K, V = wl.B, wl.K, wl.V
    np_dtype = np.uint16 if wl.dtype == "bf16" else np.float32
    target = np.empty((B, K + 1, V), dtype=np_dtype)
    draft = np.empty((B, K, V), dtype=np_dtype)
    cand = np.empty((B, K), dtype=np.int32)
    lens = make_cand_len(wl)
    if wl.sigma_n_range is not None:
        lo, hi = wl.sigma_n_range
        sig = _rng(wl.seed, "sigma").uniform(lo, hi, size=B)
    else:
        sig = np.full(B, wl.sigma_n)
    peaked = np.zeros(B, dtype=bool)
    if wl.peaked_frac > 0:
        n_peak = int(round(wl.peaked_frac * B))
        peaked[_rng(wl.seed, "peaked").permutation(B)[:n_peak]] = True

    def fill(b):
        target[b], draft[b], cand[b] = _row_logits(wl, b, int(lens[b]), float(sig[b]), bool(peaked[b]))

    threads = threads or min(32, os.cpu_count() or 1)
    if threads > 1 and B > 1:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fill, range(B)))
    else:
        for b in range(B):
            fill(b)
    uniforms = uniforms_24bit(_rng(wl.seed, "uniforms"), (B, K + 1))
    return dict(target_logits=target, draft_logits=draft, cand_tokens=cand, cand_len=lens,
                uniforms=uniforms, temperature=np.float32(wl.T), sigma_n=sig, peaked=peaked)


def make_accept_prob(wl: Workload) -> np.ndarray:
    """Stand-in head outputs ~ U(0.5, 1) for workloads that feed the stop rule directly."""
    return _rng(wl.seed, "accept_prob").uniform(0.5, 1.0, size=(wl.B, wl.K)).astype(np.float32)


def make_head_inputs(wl: Workload, weight_std: float = 0.02) -> dict:
    """Hidden states [B,K,d] ~ N(0,1) and a D-block residual head with N(0, std^2) weights,
    zero biases, all stored as bfloat16 bits."""
    assert wl.d > 0
    hidden = f32_to_bf16_bits(_rng(wl.seed, "hidden").standard_normal((wl.B, wl.K, wl.d), dtype=np.float32))
    blocks = []
    for k in range(wl.depth):
        W = _rng(wl.seed, "W", k).standard_normal((wl.d, wl.d), dtype=np.float32) * np.float32(weight_std)
        blocks.append((f32_to_bf16_bits(W), f32_to_bf16_bits(np.zeros(wl.d, np.float32))))
    w_out = f32_to_bf16_bits(_rng(wl.seed, "w_out").standard_normal(wl.d, dtype=np.float32) * np.float32(weight_std))
    return dict(hidden=hidden, blocks=blocks, w_out=w_out, b_out=np.float32(0.0), h=np.float32(wl.h))
