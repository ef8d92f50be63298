"""Sustained-rate microbenchmark of the acceptance head (Eq. 3 of arXiv 2405.19715):
`python -m paper_2405_19715_b200.headbench --rows 4096 --seconds 3`.

Runs `specdec_accept_head` (d = 4096, D = 2) back to back for a few seconds while `nvidia-smi` samples
SM clock, power draw and the power-cap flag, then does the same for a library GEMM of one block's
shape (`torch.matmul`, no epilogue), so that the head can be read against what the tensor cores
sustain under the board's power limit.  Prints one JSON line."""
from __future__ import annotations

import argparse
import json
import subprocess
import time

import numpy as np
import torch

from . import specdec, workloads as wl


def _sustain(fn, seconds: float) -> dict:
    q = "clocks.sm,power.draw,clocks_event_reasons.sw_power_cap"
    smi = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "100",
                            "-i", str(torch.cuda.current_device())], stdout=subprocess.PIPE, text=True)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0, n = time.time(), 0
    e0.record()
    while time.time() - t0 < seconds:
        for _ in range(50):
            fn()
        n += 50
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    smi.terminate()
    rows = [ln.split(",") for ln in smi.stdout.read().strip().splitlines()][3:]      # skip the ramp
    return {"ms": e0.elapsed_time(e1) / n, "sm_mhz": float(np.median([float(r[0]) for r in rows])),
            "power_w": float(np.median([float(r[1]) for r in rows])),
            "sw_power_cap": any("Active" == r[2].strip() for r in rows)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=4096, help="B*K positions (a multiple of 16)")
    ap.add_argument("--seconds", type=float, default=3.0)
    args = ap.parse_args()
    B, K = args.rows // 16, 16
    cfg = wl.CONFIGS["cfg5"].scaled(B=B, K=K)
    hd = wl.make_head_inputs(cfg)
    to = specdec.from_numpy
    hidden, w_out = to(hd["hidden"]), to(hd["w_out"])
    Ws, bs = [to(w) for w, _ in hd["blocks"]], [to(b) for _, b in hd["blocks"]]
    ctx = specdec.Context(B, K, max_d=cfg.d)
    out = torch.empty(B, K, device="cuda")
    head = _sustain(lambda: specdec.specdec_accept_head(ctx, hidden, Ws, bs, w_out, float(hd["b_out"]), out), args.seconds)
    head["tflops"] = 2.0 * cfg.depth * B * K * cfg.d * cfg.d / head["ms"] / 1e9
    a = torch.randn(B * K, cfg.d, device="cuda", dtype=torch.bfloat16)
    w = torch.randn(cfg.d, cfg.d, device="cuda", dtype=torch.bfloat16)
    gemm = _sustain(lambda: torch.matmul(a, w.t()), args.seconds)
    gemm["tflops"] = 2.0 * B * K * cfg.d * cfg.d / gemm["ms"] / 1e9
    print(json.dumps({"rows": B * K, "d": cfg.d, "depth": cfg.depth, "head": head, "library_gemm_one_block": gemm,
                      "head_vs_library": head["tflops"] / gemm["tflops"]}))


if __name__ == "__main__":
    main()
