"""Thin ctypes binding of libspecdec: argument marshalling only, every step runs in the CUDA
library.  Function names match the C ABI in include/specdec.h.  Tensors are torch CUDA
tensors (torch is used for device memory and streams only); the *_host variant takes pinned
CPU tensors.  There is no CPU fallback: a missing library or device raises.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

from . import build as _build

F32, BF16 = 0, 1
OK, EINVAL, EUNSUPPORTED, ECUDA, EDATA = 0, 1, 2, 3, 4
VERIFY_AUTO, VERIFY_DIRECT, VERIFY_STREAM, VERIFY_FUSED, VERIFY_CLUSTER = 0, 1, 2, 3, 4
DATA_BAD_LENGTH, DATA_BAD_TOKEN, DATA_WAIT_LIMIT, DATA_TOPK_TIES = 1, 2, 4, 8
VERIFY_EARLY_EXIT = 0x100

EXPORTS = ["specdec_create", "specdec_destroy", "specdec_last_error", "specdec_device_status",
           "specdec_launch_count", "specdec_last_kernel", "specdec_set_phase_stamps", "specdec_early_exit_count", "specdec_head_launch_mode", "specdec_verify_correct", "specdec_verify_correct_host",
           "specdec_accept_head", "specdec_stop", "specdec_verify_correct_static", "specdec_verify_greedy", "specdec_stop_step", "specdec_selftest_wait_limit", "specdec_verify_correct_topk", "specdec_sample",
           "specdec_shard_stats", "specdec_shard_accept", "specdec_shard_draw"]
SHARD_STATS_WIDTH, SHARD_MAX_RANKS = 8, 64
STATIC_MAX_UNITS, STATIC_MAX_V = 16384, 262144
STAMP_SLOTS = 32


class SpecdecError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"specdec error {code}: {msg}")
        self.code = code


class _Head(C.Structure):
    _fields_ = [("W", C.POINTER(C.c_void_p)), ("b", C.POINTER(C.c_void_p)), ("w_out", C.c_void_p),
                ("b_out", C.c_float), ("d", C.c_int), ("depth", C.c_int)]


class _Shard(C.Structure):
    _fields_ = [("target_logits", C.c_void_p), ("draft_logits", C.c_void_p), ("dtype", C.c_int),
                ("V_shard", C.c_int), ("v_offset", C.c_int), ("V", C.c_int)]


_lib = None


def load_library(path: str | Path | None = None) -> C.CDLL:
    """Load (building first if the sources are newer) libspecdec.so; raises if that fails."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = Path(path) if path else _build.build()
    lib = C.CDLL(str(p))
    lib.path = str(p)
    vp, ip, fp = C.c_void_p, C.c_void_p, C.c_void_p
    lib.specdec_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int, C.c_int, C.c_int]
    lib.specdec_destroy.argtypes = [C.c_void_p]
    lib.specdec_last_error.argtypes = [C.c_void_p]
    lib.specdec_last_error.restype = C.c_char_p
    lib.specdec_device_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_uint32)]
    lib.specdec_launch_count.argtypes = [C.c_void_p]
    lib.specdec_launch_count.restype = C.c_uint64
    lib.specdec_last_kernel.argtypes = [C.c_void_p]
    lib.specdec_last_kernel.restype = C.c_char_p
    lib.specdec_set_phase_stamps.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
    lib.specdec_head_launch_mode.argtypes = [C.c_void_p, C.c_int, C.c_int]
    lib.specdec_early_exit_count.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_uint64)]
    lib.specdec_verify_correct.argtypes = [C.c_void_p, vp, vp, C.c_int, ip, ip, fp, C.c_float, C.c_int, C.c_int,
                                           C.c_int, ip, ip, fp, fp, fp, C.c_uint32, C.c_void_p]
    lib.specdec_verify_correct_host.argtypes = [C.c_void_p, vp, vp, C.c_int, ip, ip, fp, C.c_float, C.c_int,
                                                C.c_int, C.c_int, ip, ip, fp, C.c_uint32, C.c_void_p]
    lib.specdec_accept_head.argtypes = [C.c_void_p, vp, C.POINTER(_Head), C.c_int, C.c_int, fp, C.c_void_p]
    lib.specdec_stop.argtypes = [C.c_void_p, fp, ip, C.c_float, C.c_int, C.c_int, ip, C.c_void_p]
    lib.specdec_verify_correct_topk.argtypes = [C.c_void_p, vp, vp, C.c_int, ip, ip, fp, C.c_float, C.c_int, C.c_int,
                                                C.c_int, C.c_int, ip, ip, fp, fp, C.c_void_p]
    lib.specdec_sample.argtypes = [C.c_void_p, vp, C.c_int, fp, C.c_float, C.c_int, C.c_int, C.c_int, ip, C.c_void_p]
    sp = C.POINTER(_Shard)
    lib.specdec_shard_stats.argtypes = [C.c_void_p, sp, ip, ip, C.c_float, C.c_int, C.c_int, fp, C.c_void_p]
    lib.specdec_shard_accept.argtypes = [C.c_void_p, sp, fp, C.c_int, ip, fp, C.c_float, C.c_int, C.c_int, ip, fp, fp,
                                         vp, C.c_void_p]
    lib.specdec_shard_draw.argtypes = [C.c_void_p, sp, fp, vp, C.c_int, C.c_int, ip, ip, fp, fp, C.c_float, C.c_int,
                                       C.c_int, ip, fp, C.c_void_p]
    lib.specdec_selftest_wait_limit.argtypes = [C.c_void_p, C.c_void_p]
    lib.specdec_stop_step.argtypes = [C.c_void_p, fp, fp, C.c_float, C.c_int, ip, C.c_void_p]
    lib.specdec_verify_greedy.argtypes = [C.c_void_p, vp, C.c_int, ip, ip, C.c_int, C.c_int, C.c_int, ip, ip, ip,
                                          C.c_void_p]
    lib.specdec_verify_correct_static.argtypes = [vp, vp, C.c_int, ip, ip, fp, C.c_float, C.c_int, C.c_int, C.c_int,
                                                  ip, ip, C.c_void_p, C.c_void_p, C.c_char_p, C.c_size_t]
    if path is None:
        _lib = lib
    return lib


def use_library(path: str | Path) -> C.CDLL:
    """Make another build of the library (the diagnostic one) the one new contexts load."""
    global _lib
    _lib = load_library(path)
    return _lib


def _ptr(t: torch.Tensor | None, dtype=None, cuda=True) -> int | None:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected {dtype}, got {t.dtype}")
    if cuda != t.is_cuda:
        raise ValueError("tensor is on the wrong side (device vs host)")
    return t.data_ptr()


def _logit_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise ValueError(f"logits must be float32 or bfloat16, got {t.dtype}")


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def from_numpy(a, device="cuda", pin: bool = False) -> torch.Tensor:
    """numpy array -> torch tensor (uint16 arrays are bfloat16 bit patterns); marshalling only."""
    import numpy as np
    a = np.ascontiguousarray(a)
    t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
    if str(device) == "cpu":
        return t.pin_memory() if pin else t
    return t.to(device)


class Context:
    """Owns a specdec_ctx.  One context serves one stream at a time."""

    def __init__(self, max_B: int, max_K: int, max_d: int = 0, device: int | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("libspecdec needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.device = torch.cuda.current_device() if device is None else device
        h = C.c_void_p()
        rc = self.lib.specdec_create(C.byref(h), self.device, max_B, max_K, max_d)
        if rc != OK:
            raise SpecdecError(rc, "specdec_create failed")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            self.lib.specdec_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            raise SpecdecError(rc, self.lib.specdec_last_error(self.handle).decode())

    def launch_count(self) -> int:
        return int(self.lib.specdec_launch_count(self.handle))

    def last_kernel(self) -> str:
        return self.lib.specdec_last_kernel(self.handle).decode()

    def set_phase_stamps(self, stamps: torch.Tensor | None):
        """specdec_set_phase_stamps of the C ABI: `stamps` is an int64 device tensor [units, STAMP_SLOTS, 2]
        (or None to switch the timestamps off); needs the diagnostic build of the library."""
        if stamps is None:
            self._check(self.lib.specdec_set_phase_stamps(self.handle, None, 0))
        else:
            self._check(self.lib.specdec_set_phase_stamps(self.handle, _ptr(stamps, torch.int64), stamps.shape[0]))

    def head_launch_mode(self, pair: bool = True, cooperative: bool = True):
        """specdec_head_launch_mode of the C ABI: rule out (False) or allow the pair-of-CTAs tiles and the single
        cooperative launch of the acceptance head for more than 256 rows."""
        self._check(self.lib.specdec_head_launch_mode(self.handle, int(pair), int(cooperative)))

    def early_exit_count(self, stream=None) -> int:
        """specdec_early_exit_count of the C ABI: logit rows left unread by early exits since the last call (synchronises)."""
        n = C.c_uint64(0)
        self._check(self.lib.specdec_early_exit_count(self.handle, _stream(stream), C.byref(n)))
        return int(n.value)

    def device_status(self, stream=None) -> int:
        """Synchronises the stream; returns the SPECDEC_DATA_* bits (0 = clean) and clears them."""
        bits = C.c_uint32(0)
        rc = self.lib.specdec_device_status(self.handle, _stream(stream), C.byref(bits))
        if rc not in (OK, EDATA):
            self._check(rc)
        return int(bits.value)


def specdec_verify_correct(ctx: Context, target_logits, draft_logits, cand_tokens, cand_len, uniforms,
                           temperature: float, n_accepted=None, next_token=None, accept_ratio=None,
                           row_stats=None, resid_mass=None, flags: int = VERIFY_AUTO, stream=None):
    """specdec_verify_correct of the C ABI.  Returns (n_accepted, next_token) device tensors
    (allocated here unless passed in)."""
    B, K1, V = target_logits.shape
    K = K1 - 1
    if tuple(draft_logits.shape) != (B, K, V) or draft_logits.dtype != target_logits.dtype:
        raise ValueError("draft_logits must be [B, K, V] of the target's dtype")
    dev = target_logits.device
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if next_token is None:
        next_token = torch.empty(B, dtype=torch.int32, device=dev)
    rc = ctx.lib.specdec_verify_correct(
        ctx.handle, _ptr(target_logits), _ptr(draft_logits), _logit_dtype(target_logits),
        _ptr(cand_tokens, torch.int32), _ptr(cand_len, torch.int32), _ptr(uniforms, torch.float32),
        float(temperature), B, K, V, _ptr(n_accepted, torch.int32), _ptr(next_token, torch.int32),
        _ptr(accept_ratio, torch.float32), _ptr(row_stats, torch.float32), _ptr(resid_mass, torch.float32),
        flags, _stream(stream))
    ctx._check(rc)
    return n_accepted, next_token


def specdec_verify_correct_host(ctx: Context, target_logits, draft_logits, cand_tokens, cand_len, uniforms,
                                temperature: float, n_accepted=None, next_token=None, accept_ratio=None,
                                flags: int = VERIFY_AUTO, stream=None):
    """specdec_verify_correct_host of the C ABI: all tensors live in (pinned) host memory; returns
    host tensors after the stream has been synchronised."""
    B, K1, V = target_logits.shape
    K = K1 - 1
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32).pin_memory()
    if next_token is None:
        next_token = torch.empty(B, dtype=torch.int32).pin_memory()
    rc = ctx.lib.specdec_verify_correct_host(
        ctx.handle, _ptr(target_logits, cuda=False), _ptr(draft_logits, cuda=False), _logit_dtype(target_logits),
        _ptr(cand_tokens, torch.int32, False), _ptr(cand_len, torch.int32, False),
        _ptr(uniforms, torch.float32, False), float(temperature), B, K, V,
        _ptr(n_accepted, torch.int32, False), _ptr(next_token, torch.int32, False),
        _ptr(accept_ratio, torch.float32, False), flags, _stream(stream))
    ctx._check(rc)
    return n_accepted, next_token


def specdec_verify_correct_topk(ctx: Context, target_logits, draft_logits, cand_tokens, cand_len, uniforms,
                                temperature: float, top_k: int, n_accepted=None, next_token=None, accept_ratio=None,
                                resid_mass=None, stream=None):
    """specdec_verify_correct_topk of the C ABI.  Returns (n_accepted, next_token) device tensors."""
    B, K1, V = target_logits.shape
    dev = target_logits.device
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if next_token is None:
        next_token = torch.empty(B, dtype=torch.int32, device=dev)
    rc = ctx.lib.specdec_verify_correct_topk(
        ctx.handle, _ptr(target_logits), _ptr(draft_logits), _logit_dtype(target_logits),
        _ptr(cand_tokens, torch.int32), _ptr(cand_len, torch.int32), _ptr(uniforms, torch.float32),
        float(temperature), int(top_k), B, K1 - 1, V, _ptr(n_accepted, torch.int32), _ptr(next_token, torch.int32),
        _ptr(accept_ratio, torch.float32), _ptr(resid_mass, torch.float32), _stream(stream))
    ctx._check(rc)
    return n_accepted, next_token


def specdec_sample(ctx: Context, logits, uniforms, temperature: float, top_k: int = 0, tokens=None, stream=None):
    """specdec_sample of the C ABI: logits [B, V], uniforms [B] -> tokens [B] int32 (device)."""
    B, V = logits.shape
    if tokens is None:
        tokens = torch.empty(B, dtype=torch.int32, device=logits.device)
    rc = ctx.lib.specdec_sample(ctx.handle, _ptr(logits), _logit_dtype(logits), _ptr(uniforms, torch.float32),
                                float(temperature), int(top_k), B, V, _ptr(tokens, torch.int32), _stream(stream))
    ctx._check(rc)
    return tokens


def _shard(target_shard, draft_shard, v_offset: int, V: int) -> _Shard:
    return _Shard(_ptr(target_shard), _ptr(draft_shard), _logit_dtype(target_shard), target_shard.shape[2],
                  int(v_offset), int(V))


def specdec_shard_stats(ctx: Context, target_shard, draft_shard, v_offset: int, V: int, cand_tokens, cand_len,
                        temperature: float, stats=None, stream=None):
    """specdec_shard_stats of the C ABI.  Returns stats [B, K+1, 8] fp32 (device)."""
    B, K1, _ = target_shard.shape
    if stats is None:
        stats = torch.empty(B, K1, SHARD_STATS_WIDTH, dtype=torch.float32, device=target_shard.device)
    sh = _shard(target_shard, draft_shard, v_offset, V)
    rc = ctx.lib.specdec_shard_stats(ctx.handle, C.byref(sh), _ptr(cand_tokens, torch.int32),
                                     _ptr(cand_len, torch.int32), float(temperature), B, K1 - 1,
                                     _ptr(stats, torch.float32), _stream(stream))
    ctx._check(rc)
    return stats


def specdec_shard_accept(ctx: Context, target_shard, draft_shard, v_offset: int, V: int, stats_all, cand_len,
                         uniforms, temperature: float, accept_ratio=None, stream=None):
    """specdec_shard_accept of the C ABI.  Returns (n_accepted [B] int32, row_norm [B, 4] fp32, mass [B] fp64)."""
    B, K1, _ = target_shard.shape
    dev = target_shard.device
    n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    row_norm = torch.empty(B, 4, dtype=torch.float32, device=dev)
    mass = torch.empty(B, dtype=torch.float64, device=dev)
    sh = _shard(target_shard, draft_shard, v_offset, V)
    rc = ctx.lib.specdec_shard_accept(ctx.handle, C.byref(sh), _ptr(stats_all, torch.float32), stats_all.shape[0],
                                      _ptr(cand_len, torch.int32), _ptr(uniforms, torch.float32), float(temperature),
                                      B, K1 - 1, _ptr(n_accepted, torch.int32), _ptr(accept_ratio, torch.float32),
                                      _ptr(row_norm, torch.float32), _ptr(mass, torch.float64), _stream(stream))
    ctx._check(rc)
    return n_accepted, row_norm, mass


def specdec_shard_draw(ctx: Context, target_shard, draft_shard, v_offset: int, V: int, stats_all, mass_all, rank: int,
                       n_accepted, cand_len, uniforms, row_norm, temperature: float, resid_mass=None, stream=None):
    """specdec_shard_draw of the C ABI.  Returns next_token [B] int32, -1 where another rank draws."""
    B, K1, _ = target_shard.shape
    next_token = torch.empty(B, dtype=torch.int32, device=target_shard.device)
    sh = _shard(target_shard, draft_shard, v_offset, V)
    rc = ctx.lib.specdec_shard_draw(ctx.handle, C.byref(sh), _ptr(stats_all, torch.float32),
                                    _ptr(mass_all, torch.float64), stats_all.shape[0], int(rank),
                                    _ptr(n_accepted, torch.int32), _ptr(cand_len, torch.int32),
                                    _ptr(uniforms, torch.float32), _ptr(row_norm, torch.float32), float(temperature),
                                    B, K1 - 1, _ptr(next_token, torch.int32), _ptr(resid_mass, torch.float32),
                                    _stream(stream))
    ctx._check(rc)
    return next_token


def specdec_selftest_wait_limit(ctx: Context, stream=None):
    """specdec_selftest_wait_limit of the C ABI (sets the WAIT_LIMIT status bit by design)."""
    ctx._check(ctx.lib.specdec_selftest_wait_limit(ctx.handle, _stream(stream)))


def specdec_stop_step(ctx: Context, accept_prob_step, p_hat, h: float, stop=None, stream=None):
    """specdec_stop_step of the C ABI: updates p_hat in place, returns stop [B] int32."""
    B = accept_prob_step.numel()
    if stop is None:
        stop = torch.empty(B, dtype=torch.int32, device=p_hat.device)
    rc = ctx.lib.specdec_stop_step(ctx.handle, _ptr(accept_prob_step, torch.float32), _ptr(p_hat, torch.float32),
                                   float(h), B, _ptr(stop, torch.int32), _stream(stream))
    ctx._check(rc)
    return stop


def specdec_verify_greedy(ctx: Context, target_logits, cand_tokens, cand_len=None, n_accepted=None, next_token=None,
                          target_argmax=None, stream=None):
    """specdec_verify_greedy of the C ABI.  Returns (n_accepted, next_token) device tensors."""
    B, K1, V = target_logits.shape
    dev = target_logits.device
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if next_token is None:
        next_token = torch.empty(B, dtype=torch.int32, device=dev)
    rc = ctx.lib.specdec_verify_greedy(ctx.handle, _ptr(target_logits), _logit_dtype(target_logits),
                                       _ptr(cand_tokens, torch.int32), _ptr(cand_len, torch.int32), B, K1 - 1, V,
                                       _ptr(n_accepted, torch.int32), _ptr(next_token, torch.int32),
                                       _ptr(target_argmax, torch.int32), _stream(stream))
    ctx._check(rc)
    return n_accepted, next_token


def specdec_accept_head(ctx: Context, hidden, W, b, w_out, b_out: float, accept_prob=None, stream=None):
    """specdec_accept_head of the C ABI.  hidden [B,K,d] bf16; W: list of [d,d] bf16; b: list of
    [d] bf16 or None entries (or None); w_out [d] bf16.  Returns accept_prob [B,K] fp32."""
    B, K, d = hidden.shape
    depth = len(W)
    Wp = (C.c_void_p * max(depth, 1))(*[_ptr(w, torch.bfloat16) for w in W])
    bl = list(b) if b is not None else [None] * depth
    bp = (C.c_void_p * max(depth, 1))(*[_ptr(x, torch.bfloat16) for x in bl])
    head = _Head(C.cast(Wp, C.POINTER(C.c_void_p)), C.cast(bp, C.POINTER(C.c_void_p)),
                 _ptr(w_out, torch.bfloat16), float(b_out), d, depth)
    if accept_prob is None:
        accept_prob = torch.empty(B, K, dtype=torch.float32, device=hidden.device)
    rc = ctx.lib.specdec_accept_head(ctx.handle, _ptr(hidden, torch.bfloat16), C.byref(head), B, K,
                                     _ptr(accept_prob, torch.float32), _stream(stream))
    ctx._check(rc)
    return accept_prob


def specdec_stop(ctx: Context, accept_prob, h: float, cand_len=None, stop_pos=None, stream=None):
    """specdec_stop of the C ABI.  Returns stop_pos [B] int32."""
    B, K = accept_prob.shape
    if stop_pos is None:
        stop_pos = torch.empty(B, dtype=torch.int32, device=accept_prob.device)
    rc = ctx.lib.specdec_stop(ctx.handle, _ptr(accept_prob, torch.float32), _ptr(cand_len, torch.int32),
                              float(h), B, K, _ptr(stop_pos, torch.int32), _stream(stream))
    ctx._check(rc)
    return stop_pos


def specdec_verify_correct_static(target_logits, draft_logits, cand_tokens, cand_len, uniforms, temperature: float,
                                  n_accepted, next_token, data_status=None, stream=None):
    """specdec_verify_correct_static of the C ABI: verify/correct without a context and without any
    allocation inside the library, for callers that may not call cudaMalloc (every device buffer,
    outputs included, is passed in).  B*(K+1) <= STATIC_MAX_UNITS and V <= STATIC_MAX_V; calls
    whose GPU work overlaps share one scratch array and race."""
    lib = load_library()
    B, K1, V = target_logits.shape
    err = C.create_string_buffer(256)
    rc = lib.specdec_verify_correct_static(
        _ptr(target_logits), _ptr(draft_logits), _logit_dtype(target_logits), _ptr(cand_tokens, torch.int32),
        _ptr(cand_len, torch.int32), _ptr(uniforms, torch.float32), float(temperature), B, K1 - 1, V,
        _ptr(n_accepted, torch.int32), _ptr(next_token, torch.int32),
        None if data_status is None else data_status.data_ptr(), _stream(stream), err, len(err))
    if rc != OK:
        raise SpecdecError(rc, err.value.decode())
    return n_accepted, next_token
