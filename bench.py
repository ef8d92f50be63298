#!/usr/bin/env python
"""Benchmark of the SpecDec++ hot path on B200: head -> stop rule -> verify/correct.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4]

One step is one pass of the whole hot path over one batch of synthetic input.  Prints ONE JSON
line (rank 0).  `value` is candidate tokens verified per second with inputs resident in HBM;
`e2e` is the same metric through the host-buffer entry point (host->device copy of every input
and device->host copy of the results inside the timed region).  For N > 1 the batch rows are
sharded (each rank owns its own rows, no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2405_19715_b200 import workloads as wl  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of one verify/correct launch (the kernel the library picks at this
# size), from the ncu capture at half the batch summarised in profiles/verify_direct_cfg4_B128.md, scaled by units.
NCU_TRAFFIC_BYTES = {"cfg4": 2.3044e9}

METRIC = "verified candidate tokens/s"
UNIT = "tokens/s"


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_config(cfg: wl.Workload, rank: int) -> wl.Workload:
    """Rank r owns its own batch rows (weak scaling): same shapes, a row stream of its own."""
    return cfg.scaled(seed=cfg.seed + rank)


def aggregate(elapsed_ms: float, tokens: float, world: int, device):
    """Whole-job numbers: the slowest rank's time and the tokens all ranks verified."""
    return max_over_ranks(elapsed_ms, world, device), sum_over_ranks(tokens, world, device)


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def algorithmic_bytes(cfg: wl.Workload, lens: np.ndarray) -> int:
    """Every logit the method needs, once: (2 L_b + 1) rows of V elements per batch row."""
    es = 2 if cfg.dtype == "bf16" else 4
    return int((2 * lens.astype(np.int64) + 1).sum()) * cfg.V * es


# ----------------------------------------------------------------------------------------- CPU arm
def oracle_sample_rate(cfg: wl.Workload, inp: dict, budget_s: float, head=None, top_k=None):
    """Times the CPU oracle (as it stands) on leading batch rows until `budget_s` is used.
    Returns (tokens/s, rows used, seconds, threads)."""
    from oracle import specdec_oracle as orc
    lens = inp["cand_len"]
    t0 = time.perf_counter()
    rows = tokens = 0
    chunk = 4
    while rows < cfg.B and time.perf_counter() - t0 < budget_s:
        sl = slice(rows, min(rows + chunk, cfg.B))
        if head is not None:
            a = orc.accept_head(head["hidden"][sl], head["blocks"], head["w_out"], float(head["b_out"]))
            orc.stop_rule(a.astype(np.float32), cfg.h, lens[sl])
        orc.verify_correct(inp["target_logits"][sl], inp["draft_logits"][sl], inp["cand_tokens"][sl], lens[sl],
                           inp["uniforms"][sl], inp["temperature"], top_k=top_k)
        tokens += int(lens[sl].sum())
        rows = sl.stop
    dt = time.perf_counter() - t0
    return tokens / dt, rows, dt, 1      # numpy's exp / cumsum run on one thread


def run_reference(args, cfg):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    sub = cfg.scaled(B=min(cfg.B, 8))          # bounded sample: the first rows of the workload
    inp = wl.make_verify_inputs(sub)
    hd = wl.make_head_inputs(wl.CONFIGS["cfg5"].scaled(B=sub.B, K=sub.K, seed=sub.seed))
    rates = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        from oracle import specdec_oracle as orc
        a = orc.accept_head(hd["hidden"], hd["blocks"], hd["w_out"], float(hd["b_out"]))
        orc.stop_rule(a.astype(np.float32), sub.h, inp["cand_len"])
        orc.verify_correct(inp["target_logits"], inp["draft_logits"], inp["cand_tokens"], inp["cand_len"],
                           inp["uniforms"], inp["temperature"])
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            rates.append(dt)
    ms = 1e3 * float(np.mean(rates))
    tokens = int(inp["cand_len"].sum())
    value = tokens / (ms * 1e-3)
    sample = f"first {sub.B} of {cfg.B} batch rows of {cfg.name} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": workload_config(cfg, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg: wl.Workload, world: int) -> dict:
    return {"workload": f"{cfg.name}: acceptance head (d=4096, D=2) on B*K positions -> stop rule -> verify/correct, "
                        f"B={cfg.B} K={cfg.K} V={cfg.V} {cfg.dtype} T={cfg.T} (per GPU)",
            "B_per_gpu": cfg.B, "K": cfg.K, "V": cfg.V, "logit_dtype": cfg.dtype, "sharding": f"batch rows x{world}",
            "l2": "inputs exceed L2 (no flush needed)" if cfg.B * (2 * cfg.K + 1) * cfg.V * 2 > 2 * 126e6
                  else "rotating input copies > 2x L2"}


# ----------------------------------------------------------------------------------------- GPU arm
def run_ours(args, cfg):
    from paper_2405_19715_b200 import specdec
    to_torch = specdec.from_numpy
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    cfg = shard_config(cfg, rank)
    inp = wl.make_verify_inputs(cfg)
    lens_np = inp["cand_len"]
    es = 2 if cfg.dtype == "bf16" else 4
    per_copy = cfg.B * (2 * cfg.K + 1) * cfg.V * es
    copies = 1 if per_copy > 2 * 126e6 else int(np.ceil(2 * 126e6 / per_copy)) + 1

    host = {k: to_torch(np.ascontiguousarray(inp[k]), "cpu", pin=True)
            for k in ("target_logits", "draft_logits", "cand_tokens", "cand_len", "uniforms")}
    devs = [{k: v.to(dev) for k, v in host.items()} for _ in range(copies)]
    # acceptance head of the cfg5 recipe (d = 4096, D = 2, N(0, 0.02^2) weights) on this batch's B x K positions
    hcfg = wl.CONFIGS["cfg5"].scaled(B=cfg.B, K=cfg.K, seed=cfg.seed)
    hd = wl.make_head_inputs(hcfg)
    hidden = to_torch(hd["hidden"]).to(dev)
    Ws = [to_torch(w).to(dev) for w, _ in hd["blocks"]]
    bs = [to_torch(b).to(dev) for _, b in hd["blocks"]]
    w_out = to_torch(hd["w_out"]).to(dev)
    head_prob = torch.empty(cfg.B, cfg.K, dtype=torch.float32, device=dev)
    ctx = specdec.Context(cfg.B, cfg.K, max_d=hcfg.d)
    n_out = torch.empty(cfg.B, dtype=torch.int32, device=dev)
    t_out = torch.empty(cfg.B, dtype=torch.int32, device=dev)
    stop_pos = torch.empty(cfg.B, dtype=torch.int32, device=dev)
    T = float(inp["temperature"])

    def step(i, ev=None):
        d = devs[i % copies]
        if ev:
            ev[2].record()
        specdec.specdec_accept_head(ctx, hidden, Ws, bs, w_out, float(hd["b_out"]), head_prob)
        if ev:
            ev[3].record()
        specdec.specdec_stop(ctx, head_prob, cfg.h, d["cand_len"], stop_pos)
        if ev:
            ev[0].record()
        if args.top_k > 0:
            specdec.specdec_verify_correct_topk(ctx, d["target_logits"], d["draft_logits"], d["cand_tokens"],
                                                d["cand_len"], d["uniforms"], T, args.top_k, n_out, t_out)
        else:
            specdec.specdec_verify_correct(ctx, d["target_logits"], d["draft_logits"], d["cand_tokens"], d["cand_len"],
                                           d["uniforms"], T, n_out, t_out, flags=args.kernel)
        if ev:
            ev[1].record()

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    launches0 = ctx.launch_count()
    evs = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(4)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    torch.cuda.synchronize()
    e0.record()
    for i in range(args.steps):
        step(i, evs[i])
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    launches = ctx.launch_count() - launches0
    elapsed_ms, tokens_step = aggregate(e0.elapsed_time(e1), float(lens_np.sum()), world, dev)
    clocks = sampler.stop() if rank == 0 else None
    verify_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    head_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
    stop_ms = float(np.mean([e[3].elapsed_time(e[0]) for e in evs]))
    ms_per_step = elapsed_ms / args.steps
    value = tokens_step / (ms_per_step * 1e-3)

    # end to end through the host-buffer entry point (pinned host inputs, results back on the host)
    e2e_steps = max(1, min(args.steps, 5))
    h_n = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    h_t = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    h_stop = torch.empty(cfg.B, dtype=torch.int32).pin_memory()

    h_hidden = to_torch(hd["hidden"], "cpu", pin=True)

    def e2e_step():
        hh = h_hidden.to(dev, non_blocking=True)
        l = host["cand_len"].to(dev, non_blocking=True)
        specdec.specdec_accept_head(ctx, hh, Ws, bs, w_out, float(hd["b_out"]), head_prob)
        specdec.specdec_stop(ctx, head_prob, cfg.h, l, stop_pos)
        h_stop.copy_(stop_pos, non_blocking=True)
        specdec.specdec_verify_correct_host(ctx, host["target_logits"], host["draft_logits"], host["cand_tokens"],
                                            host["cand_len"], host["uniforms"], T, h_n, h_t, flags=args.kernel)

    if args.no_e2e or args.top_k > 0:               # the host-buffer entry point has no top-k form
        e2e_steps = 0
        e2e_ms = float("nan")
    else:
        e2e_step()
        torch.cuda.synchronize()
        barrier(world)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / e2e_steps
    h2d = (sum(v.numel() * v.element_size() for v in host.values()) + h_hidden.numel() * 2
           + host["cand_len"].numel() * 4)
    d2h = 3 * cfg.B * 4

    if rank != 0:
        return
    peaks = measured_peaks()
    alg = algorithmic_bytes(cfg, lens_np)
    head_flops = 2.0 * hcfg.depth * cfg.B * cfg.K * hcfg.d * hcfg.d
    achieved = alg / (verify_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, world),
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": tokens_step / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms},
        "roofline": {"kernel": "verify/correct", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                     "frac_of_nominal_8TBs": achieved / 8000.0, "algorithmic_bytes": alg, "kernel_ms": verify_ms,
                     "traffic": NCU_TRAFFIC_BYTES.get(cfg.name) if args.kernel == 0 and args.top_k == 0 else None},
        "parts_ms": {"head": head_ms, "stop": stop_ms, "verify": verify_ms},
        "roofline_head": {"kernel": "acceptance head (2 x [M,4096]x[4096,4096] bf16 GEMM)", "bound": "tensor",
                          "achieved": head_flops / (head_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"],
                          "unit": "TFLOP/s", "frac": head_flops / (head_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                          "peak_source": peaks["source"] + " cuBLAS bf16 (sustained)"},
    }
    if args.top_k > 0:
        line["config"]["top_k"] = args.top_k
        line["roofline"]["kernel"] = f"verify/correct, top-k {args.top_k}"
        line["e2e"] = None
    if world == 1 and not args.no_cpu_baseline:
        rate, rows, dt, cores = oracle_sample_rate(cfg, inp, args.cpu_budget, hd, args.top_k or None)
        line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {rows} of {cfg.B} batch rows of {cfg.name}, {dt:.1f} s"}
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(wl.CONFIGS))
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 one CTA per unit, 2 two-launch TMA pipeline, 3 fused TMA pipeline, 4 cluster per unit")
    ap.add_argument("--top-k", type=int, default=0,
                    help="verify under top-k sampling (the paper's runs use 50); 0 = whole vocabulary, the headline workload")
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling runs)")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.workload]
    if args.batch:
        cfg = cfg.scaled(B=args.batch, name=f"{cfg.name}(B={args.batch})")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
