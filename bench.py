#!/usr/bin/env python
"""Benchmark of the SpecDec++ hot path on B200: head -> stop rule -> verify/correct.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4]
                    [--vocab-shards] [--top-k 50]

One step is one pass of the whole hot path over one batch of synthetic input.  Prints ONE JSON
line (rank 0).  `value` is candidate tokens verified per second with inputs resident in HBM;
`e2e` is the same metric through the host-buffer entry point (host->device copy of every input
and device->host copy of the results inside the timed region); `sustained` repeats the step back
to back for a couple of seconds with clocks and power sampled.

Several GPUs: `python bench.py --gpus N` starts N ranks by itself (one process per GPU through
torch.distributed.run on 127.0.0.1); under an external torchrun it joins the ranks it is given.
Batch rows are independent, so every rank verifies rows of its own and nothing of the data path
crosses GPUs (weak scaling).  `--vocab-shards` instead splits the vocabulary of ONE batch over the
ranks (the target model sharded over GPUs) and times the sharded verify/correct with its three
small collectives (strong scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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

METRIC = "verified candidate tokens/s"
UNIT = "tokens/s"
TRAFFIC_FILE = ROOT / "profiles" / "dram_traffic.json"


def measured_peaks():
    """Roofline denominators: measured on this machine's B200s when the file is there, else the fallback."""
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_burst=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def ncu_traffic(kernel: str, units: int):
    """DRAM read + write bytes of one launch from the ncu capture recorded for `kernel`, scaled by the
    (row, position) units processed (traffic grows in proportion to them); None when no capture of the
    current kernel is on record."""
    if not TRAFFIC_FILE.exists():
        return None
    rec = json.loads(TRAFFIC_FILE.read_text()).get(kernel)
    if not rec or not rec.get("current", False):
        return None
    return float(rec["dram_bytes"]) * units / float(rec["units"])


class ClockSampler:
    """Samples SM clocks, power and throttle reasons with nvidia-smi while a timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 100):
        self.gpu = gpu_index
        self.period_ms = period_ms
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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
        sm, pw, mx, reasons = [], [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
                pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "power_w_median": float(np.median(pw)) if pw else None,
                "power_w_max": float(np.max(pw)) if pw else None}


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


def algorithmic_bytes(cfg: wl.Workload, lens: np.ndarray, V: int | None = None) -> int:
    """Every logit the method needs, once: (2 L_b + 1) rows of V elements per batch row."""
    es = 2 if cfg.dtype == "bf16" else 4
    return int((2 * lens.astype(np.int64) + 1).sum()) * (cfg.V if V is None else V) * es


# ----------------------------------------------------------------------------------------- launcher
def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n: int, argv: list[str], extra_env: dict | None = None) -> tuple[int, str]:
    """Start n ranks of this script on this node (one process per GPU, rendezvous on 127.0.0.1) and
    return (exit code, what rank 0 printed).  NCCL's own log stays on so that its communicator lines
    show the n ranks."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.update(extra_env or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), str(ROOT / "bench.py"), *argv]
    proc = subprocess.run(cmd, stdout=subprocess.PIPE, text=True, env=env)
    return proc.returncode, proc.stdout


def run_stub(args):
    """The launcher's self-check: ranks that meet over gloo on the CPU, run a step that does nothing,
    and report through the same reductions as the real benchmark."""
    import torch.distributed as dist
    rank, world, _ = dist_env()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dev = torch.device("cpu")
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.001)
    ms, tokens = aggregate(1e3 * (time.perf_counter() - t0), 10.0 * (rank + 1), world, dev)
    seen = [None] * world
    dist.all_gather_object(seen, (rank, world))
    barrier(world)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "stub": True, "tokens_per_step": tokens, "ranks_seen": seen}), flush=True)
    dist.destroy_process_group()


# ----------------------------------------------------------------------------------------- CPU arm
def _oracle_rows(inp: dict, cfg: wl.Workload, rows: slice, head=None, top_k=None) -> int:
    from oracle import specdec_oracle as orc
    lens = inp["cand_len"]
    if head is not None:
        a = orc.accept_head(head["hidden"][rows], head["blocks"], head["w_out"], float(head["b_out"]))
        orc.stop_rule(a.astype(np.float32), cfg.h, lens[rows])
    orc.verify_correct(inp["target_logits"][rows], inp["draft_logits"][rows], inp["cand_tokens"][rows], lens[rows],
                       inp["uniforms"][rows], inp["temperature"], top_k=top_k)
    return int(lens[rows].sum())


def _one_thread():
    """Numerical libraries limited to one thread (numpy's own loops are single-threaded, its BLAS is not)."""
    from threadpoolctl import threadpool_limits
    return threadpool_limits(limits=1)


def oracle_sample_rate(cfg: wl.Workload, inp: dict, budget_s: float, head=None, top_k=None):
    """Times the CPU oracle (as it stands) on the leading batch rows that fit `budget_s`, on one
    thread: one call for the whole sample.  Returns (tokens/s, rows used, seconds)."""
    with _one_thread():
        t0 = time.perf_counter()
        _oracle_rows(inp, cfg, slice(0, min(2, cfg.B)), None, top_k)          # sizes the sample, not reported
        per_row = (time.perf_counter() - t0) / min(2, cfg.B)
        rows = int(min(cfg.B, max(2, budget_s * 0.8 / per_row)))
        t0 = time.perf_counter()
        tokens = _oracle_rows(inp, cfg, slice(0, rows), head, top_k)
        dt = time.perf_counter() - t0
    return tokens / dt, rows, dt


_POOL_STATE = None


def _pool_task(rows):
    inp, cfg, head, top_k = _POOL_STATE
    with _one_thread():
        return _oracle_rows(inp, cfg, slice(*rows), head, top_k)


def usable_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_all_cores_rate(cfg: wl.Workload, inp: dict, budget_s: float, rate_one_core: float, head=None, top_k=None):
    """The same oracle with the batch rows (independent problems) spread over all host cores: forked
    workers that inherit the inputs, one contiguous row range each, one thread each.  Returns
    (tokens/s, rows used, seconds, cores)."""
    import multiprocessing as mp
    global _POOL_STATE
    cores = usable_cores()
    tokens_per_row = float(inp["cand_len"].mean()) or 1.0
    rows = int(min(cfg.B, max(cores, np.ceil(rate_one_core / tokens_per_row * cores * budget_s * 0.6))))
    per = -(-rows // cores)
    tasks = [(r, min(r + per, rows)) for r in range(0, rows, per)]
    _POOL_STATE = (inp, cfg, head, top_k)
    try:
        with mp.get_context("fork").Pool(cores) as pool:
            pool.map(abs, range(4 * cores))                        # workers up before the clock starts
            t0 = time.perf_counter()
            tokens = sum(pool.map(_pool_task, tasks, chunksize=1))
            dt = time.perf_counter() - t0
    finally:
        _POOL_STATE = None
    return tokens / dt, rows, dt, cores


def run_reference(args, cfg):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the workload per step."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    sub = cfg.scaled(B=min(cfg.B, 8))          # bounded sample: the first rows of the workload
    inp = wl.make_verify_inputs(sub)
    hd = wl.make_head_inputs(wl.CONFIGS["cfg5"].scaled(B=sub.B, K=sub.K, seed=sub.seed))
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        _oracle_rows(inp, sub, slice(0, sub.B), hd)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * float(np.mean(times))
    tokens = int(inp["cand_len"].sum())
    value = tokens / (ms * 1e-3)
    sample = f"first {sub.B} of {cfg.B} batch rows of {cfg.name} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": workload_config(cfg, max(world, 1)),
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
def init_dist(world: int, dev):
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)


def run_ours(args, cfg):
    from paper_2405_19715_b200 import specdec
    to_torch = specdec.from_numpy
    rank, world, local = dist_env()
    cfg = shard_config(cfg, rank)
    inp = wl.make_verify_inputs(cfg)
    lens_np = inp["cand_len"]
    # The oracle is timed first, before this process touches the GPU: its all-cores leg forks workers,
    # and a process forked after CUDA has been initialised is not safe to run.
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        hd0 = wl.make_head_inputs(wl.CONFIGS["cfg5"].scaled(B=cfg.B, K=cfg.K, seed=cfg.seed))
        rate, rows, dt = oracle_sample_rate(cfg, inp, args.cpu_budget, hd0, args.top_k or None)
        cpu_baseline = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": f"first {rows} of {cfg.B} batch rows of {cfg.name}, {dt:.1f} s"}
        try:
            rate_n, rows_n, dt_n, cores = oracle_all_cores_rate(cfg, inp, args.cpu_budget, rate, hd0, args.top_k or None)
            cpu_baseline["all_cores"] = {
                "value": rate_n, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"first {rows_n} of {cfg.B} batch rows of {cfg.name} over {cores} forked workers, {dt_n:.1f} s"}
        except Exception as e:                       # the single-core figure stands on its own
            cpu_baseline["all_cores"] = {"unavailable": repr(e)}
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    init_dist(world, dev)
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

    def parts(evs):
        return (float(np.mean([e[2].elapsed_time(e[3]) for e in evs])), float(np.mean([e[3].elapsed_time(e[0]) for e in evs])),
                float(np.mean([e[0].elapsed_time(e[1]) for e in evs])))

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
    head_ms, stop_ms, verify_ms = parts(evs)
    ms_per_step = elapsed_ms / args.steps
    value = tokens_step / (ms_per_step * 1e-3)

    # the same step back to back for a couple of seconds: the power-capped regime
    sustained = None
    if args.sustained_seconds > 0:
        n_sus = int(max(50, np.ceil(args.sustained_seconds * 1e3 / ms_per_step)))
        every = max(1, n_sus // 64)
        sus_evs = []
        sampler2 = ClockSampler(local, period_ms=50)
        if rank == 0:
            sampler2.start()
            time.sleep(0.1)
        barrier(world)
        torch.cuda.synchronize()
        e0.record()
        for i in range(n_sus):
            if i % every == 0 and i > n_sus // 4:      # per-part times from the settled part of the loop
                ev = tuple(torch.cuda.Event(enable_timing=True) for _ in range(4))
                sus_evs.append(ev)
                step(i, ev)
            else:
                step(i)
        e1.record()
        torch.cuda.synchronize()
        sus_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / n_sus
        ck = sampler2.stop() if rank == 0 else None
        h_ms, s_ms, v_ms = parts(sus_evs)
        mhz = (ck or {}).get("sm_mhz")
        sustained = {"seconds": sus_ms * n_sus * 1e-3, "steps": n_sus, "ms_per_step": sus_ms,
                     "value": tokens_step / (sus_ms * 1e-3), "unit": UNIT, "clocks": ck,
                     "parts_ms": {"head": h_ms, "stop": s_ms, "verify": v_ms},
                     "ms_times_mhz": None if not mhz else {"head": h_ms * mhz, "verify": v_ms * mhz},
                     "burst_ms_times_mhz": None if not clocks or not clocks.get("sm_mhz") else
                     {"head": head_ms * clocks["sm_mhz"], "verify": verify_ms * clocks["sm_mhz"]}}

    # the same verify/correct call on ONE copy of the inputs, back to back: where a workload fits in L2 this is
    # the warm figure (inputs served from L2), reported beside the cold one of the timed region
    warm_ms = None
    if copies > 1 and args.top_k == 0 and not args.no_extras:
        d0 = devs[0]
        def warm_call():
            specdec.specdec_verify_correct(ctx, d0["target_logits"], d0["draft_logits"], d0["cand_tokens"], d0["cand_len"],
                                           d0["uniforms"], T, n_out, t_out, flags=args.kernel)
        for _ in range(5):
            warm_call()
        wev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        torch.cuda.synchronize()
        wev[0].record()
        for i in range(args.steps):
            warm_call()
            wev[i + 1].record()
        torch.cuda.synchronize()
        warm_ms = float(np.mean([wev[i].elapsed_time(wev[i + 1]) for i in range(args.steps)]))

    # Not the contract's path, reported beside it: the call with SPECDEC_VERIFY_EARLY_EXIT (units that start after
    # an earlier position of their row has been rejected read nothing; outputs identical), cold inputs
    early = None
    if args.top_k == 0 and not args.no_extras:
        def early_call(i):
            d = devs[i % copies]
            specdec.specdec_verify_correct(ctx, d["target_logits"], d["draft_logits"], d["cand_tokens"], d["cand_len"],
                                           d["uniforms"], T, n_out, t_out, flags=args.kernel | specdec.VERIFY_EARLY_EXIT)
        for i in range(3):
            early_call(i)
        ctx.early_exit_count()
        eev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        eev[0].record()
        for i in range(args.steps):
            early_call(i)
            eev[i + 1].record()
        torch.cuda.synchronize()
        rows_unread = ctx.early_exit_count() / args.steps
        early_ms = float(np.mean([eev[i].elapsed_time(eev[i + 1]) for i in range(args.steps)]))
        early = {"kernel_ms": early_ms, "logit_rows_not_read_per_call": rows_unread, "kernel": ctx.last_kernel()}

    # Short steps: the same launches replayed from a CUDA graph, so that no host work sits between them (with
    # three library calls per step the host needs tens of microseconds, more than these steps take on the GPU).
    # A graph holds one step per input copy, so the logits are as cold as in the timed region.
    graph_times = None
    if ms_per_step < 0.3 and args.top_k == 0 and world == 1 and not args.no_extras:
        n_g = max(copies, 8)

        def head_call(i):
            specdec.specdec_accept_head(ctx, hidden, Ws, bs, w_out, float(hd["b_out"]), head_prob)

        def stop_call(i):
            specdec.specdec_stop(ctx, head_prob, cfg.h, devs[i % copies]["cand_len"], stop_pos)

        def verify_call(i):
            d = devs[i % copies]
            specdec.specdec_verify_correct(ctx, d["target_logits"], d["draft_logits"], d["cand_tokens"], d["cand_len"],
                                           d["uniforms"], T, n_out, t_out, flags=args.kernel)

        def replayed_ms(fn):
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(n_g):
                    fn(i)
            g.replay()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(5):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / (5 * n_g)

        try:
            graph_times = {"ms_per_step": replayed_ms(lambda i: step(i)),
                           "parts_ms": {"head": replayed_ms(head_call), "stop": replayed_ms(stop_call), "verify": replayed_ms(verify_call)},
                           "note": "launches replayed from a CUDA graph (no host in the loop); logits cold, head weights "
                                   "as in the step (they stay in L2 between steps); each part replayed on its own"}
        except Exception as e:                       # the event-timed figures stand on their own
            graph_times = {"unavailable": repr(e)}
        assert ctx.device_status() == 0

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

    if rank == 0:
        peaks = measured_peaks()
        alg = algorithmic_bytes(cfg, lens_np)
        units = int((lens_np.astype(np.int64) + 1).sum())
        head_flops = 2.0 * hcfg.depth * cfg.B * cfg.K * hcfg.d * hcfg.d
        achieved = alg / (verify_ms * 1e-3) / 1e9
        kernel_name = ctx.last_kernel()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, world),
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": tokens_step / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms},
            "roofline": {"kernel": f"verify/correct ({kernel_name})", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                         "frac_of_nominal_8TBs": achieved / 8000.0, "algorithmic_bytes": alg, "kernel_ms": verify_ms,
                         "traffic": ncu_traffic(f"{kernel_name}<{cfg.dtype}>", units),
                         "cache": "cold: every step reads its logits from HBM",
                         "warm": None if warm_ms is None else
                         {"kernel_ms": warm_ms, "achieved": alg / (warm_ms * 1e-3) / 1e9, "unit": "GB/s",
                          "note": "same call repeated on one copy of the inputs (served from L2 where they fit); not a DRAM figure"}},
            "parts_ms": {"head": head_ms, "stop": stop_ms, "verify": verify_ms},
            "graph_replay": graph_times,
            "early_exit": None if early is None else dict(
                early, bytes_read=alg - early["logit_rows_not_read_per_call"] * cfg.V * es,
                achieved_read_gbs=(alg - early["logit_rows_not_read_per_call"] * cfg.V * es) / (early["kernel_ms"] * 1e-3) / 1e9,
                tokens_per_s_verify_only=tokens_step / (early["kernel_ms"] * 1e-3),
                note="SPECDEC_VERIFY_EARLY_EXIT: positions after a row's first rejection are not read when that rejection is "
                     "already known; same n_accepted / next_token; not part of value, roofline or e2e above"),
            # the timed region lasts milliseconds at full clocks: the burst peak is its denominator;
            # the power-capped loop is measured against the sustained one
            "roofline_head": {"kernel": "acceptance head (2 x [M,4096]x[4096,4096] bf16 GEMM)", "bound": "tensor",
                              "achieved": head_flops / (head_ms * 1e-3) / 1e12, "peak": peaks["bf16_burst"],
                              "unit": "TFLOP/s", "frac": head_flops / (head_ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                              "peak_source": peaks["source"] + " cuBLAS bf16 (burst)"},
        }
        if sustained is not None:
            sh = head_flops / (sustained["parts_ms"]["head"] * 1e-3) / 1e12
            sv = alg / (sustained["parts_ms"]["verify"] * 1e-3) / 1e9
            sustained["roofline_head"] = {"achieved": sh, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                                          "frac": sh / peaks["bf16_sustained"], "peak_source": peaks["source"] + " cuBLAS bf16 (sustained)"}
            sustained["roofline"] = {"achieved": sv, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": sv / peaks["hbm_gbs"]}
            line["sustained"] = sustained
        if args.top_k > 0:
            line["config"]["top_k"] = args.top_k
            line["e2e"] = None
        if args.early_exit:
            line["config"]["early_exit"] = ("timed step run with SPECDEC_VERIFY_EARLY_EXIT: roofline.achieved still divides the "
                                            "algorithmic bytes of all needed rows by the call time, so it can exceed the peak")
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


PHASES = [("CTA start -> length known", 0, 1), ("length known -> scalars requested", 1, 10),
          ("scalars requested -> first thread's share of the statistics pass done", 10, 2),
          ("first thread done -> warps' sums merged by warp 0 (waits for the CTA's slowest warp)", 2, 11),
          ("log-probabilities and ratio", 11, 12), ("flag and optional outputs stored", 12, 13),
          ("earlier flags looked up, normalisers", 13, 4), ("decision -> seen by the CTA", 4, 5),
          ("draw: slab sums", 5, 6), ("draw: prefix, slab walk", 6, 7), ("no draw: decision -> arrival", 5, 7),
          ("arrival counted on the row", 7, 8), ("last arriver: ballot + outputs", 8, 9), ("whole unit", 0, 9)]


def run_phases(args, cfg):
    """Per-phase device timestamps of the one-CTA-per-unit verify/correct kernel on `cfg` (cold inputs): builds
    and loads the diagnostic library (-DSPECDEC_STAMPS) and prints a markdown table.  Not a benchmark line."""
    from paper_2405_19715_b200 import build as libbuild, specdec
    specdec.use_library(libbuild.build(stamps=True))
    to_torch = specdec.from_numpy
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    inp = wl.make_verify_inputs(cfg)
    es = 2 if cfg.dtype == "bf16" else 4
    per_copy = cfg.B * (2 * cfg.K + 1) * cfg.V * es
    copies = 1 if per_copy > 2 * 126e6 else int(np.ceil(2 * 126e6 / per_copy)) + 1
    base = {k: to_torch(np.ascontiguousarray(inp[k]), "cpu") for k in ("target_logits", "draft_logits", "cand_tokens", "cand_len", "uniforms")}
    devs = [{k: v.to(dev) for k, v in base.items()} for _ in range(copies)]
    ctx = specdec.Context(cfg.B, cfg.K)
    units = cfg.B * (cfg.K + 1)
    stamps = torch.zeros(units, specdec.STAMP_SLOTS, 2, dtype=torch.int64, device=dev)
    n_out = torch.empty(cfg.B, dtype=torch.int32, device=dev)
    t_out = torch.empty(cfg.B, dtype=torch.int32, device=dev)
    T = float(inp["temperature"])
    kernel = args.kernel or specdec.VERIFY_DIRECT

    def call(i):
        d = devs[i % copies]
        specdec.specdec_verify_correct(ctx, d["target_logits"], d["draft_logits"], d["cand_tokens"], d["cand_len"],
                                       d["uniforms"], T, n_out, t_out, flags=kernel)
    for i in range(max(args.warmup, 3)):
        call(i)
    torch.cuda.synchronize()
    ctx.set_phase_stamps(stamps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    durs = {name: [] for name, _, _ in PHASES}
    done_at, start_at, ev_ms, span, mhz, skew, wait0 = [], [], [], [], [], [], []
    for i in range(args.steps):
        stamps.zero_()
        e0.record()
        call(i)
        e1.record()
        torch.cuda.synchronize()
        ev_ms.append(e0.elapsed_time(e1))
        st = stamps.cpu().numpy()
        g, c = st[:, :, 0].astype(np.float64), st[:, :, 1].astype(np.float64)
        live = g[:, 9] > 0
        t0 = g[live, 0].min()
        start_at.append(np.sort(g[live, 0] - t0) * 1e-3)
        done_at.append(np.sort(g[live, 9] - t0) * 1e-3)
        span.append((g[live, 9].max() - t0) * 1e-3)
        # durations inside a unit from the SM's cycle counter (the global timer ticks too coarsely for them),
        # converted with the cycles per nanosecond seen over whole units
        ghz = float(np.median((c[live, 9] - c[live, 0]) / np.maximum(g[live, 9] - g[live, 0], 1.0)))
        mhz.append(1e3 * ghz)
        for name, a, b in PHASES:
            ok = live & (c[:, a] > 0) & (c[:, b] > 0)
            if name.startswith("no draw"):
                ok &= c[:, 6] == 0
            durs[name].append((c[ok, b] - c[ok, a]) / ghz * 1e-3)
        wdone = np.where(c[live, 16:32] > 0, c[live, 16:32], np.nan)
        skew.append((np.nanmax(wdone, 1) - np.nanmin(wdone, 1)) / ghz * 1e-3)
        wait0.append((c[live, 11] - c[live, 16]) / ghz * 1e-3)
    q = lambda x, p: float(np.percentile(x, p)) if len(x) else float("nan")
    print(f"workload {cfg.name}: B={cfg.B} K={cfg.K} V={cfg.V} {cfg.dtype}, kernel {ctx.last_kernel()}, {args.steps} cold calls; "
          f"phase durations in us from the SM cycle counters ({np.median(mhz):.0f} MHz), unit start / finish times from the device's global timer")
    print(f"call by CUDA events: mean {1e3 * np.mean(ev_ms):.1f} us; first CTA start -> last unit end: mean {np.mean(span):.1f} us")
    print("| phase | units per call | median | p10 | p90 | max |\n|---|---|---|---|---|---|")
    for name, _, _ in PHASES:
        x = np.concatenate(durs[name])
        print(f"| {name} | {len(x) // args.steps} | {q(x, 50):.2f} | {q(x, 10):.2f} | {q(x, 90):.2f} | {q(x, 100):.2f} |")
    for name, x in (("first warp's statistics done -> last warp's (skew inside the CTA)", np.concatenate(skew)),):
        print(f"| {name} | {len(x) // args.steps} | {q(x, 50):.2f} | {q(x, 10):.2f} | {q(x, 90):.2f} | {q(x, 100):.2f} |")
    sa, da = np.mean(np.stack(start_at), 0), np.mean(np.stack(done_at), 0)
    n = len(sa)
    print("| unit rank | started at | finished at |\n|---|---|---|")
    for f in (0.0, 0.25, 0.5, 0.75, 0.9, 0.97, 1.0):
        k = min(n - 1, int(round(f * (n - 1))))
        print(f"| {k + 1} of {n} | {sa[k]:.1f} | {da[k]:.1f} |")
    ctx.set_phase_stamps(None)
    ctx.close()


def run_head_phases(args):
    """Phase timestamps of one CTA of the weights-as-M head kernel (17 to 256 rows) for one cold call of the
    acceptance head with d = 4096, D = 2 and --batch rows (default 64): diagnostic build, not a benchmark line."""
    import ctypes
    from paper_2405_19715_b200 import build as libbuild, specdec
    lib = specdec.use_library(libbuild.build(stamps=True))
    torch.cuda.set_device(0)
    M, d, D, copies = args.batch or 64, 4096, 2, 6
    g = torch.Generator(device="cuda").manual_seed(1)
    Ws = [[(torch.randn(d, d, device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(D)] for _ in range(copies)]
    w_out = (torch.randn(d, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    ctx = specdec.Context(M, 1, max_d=d)
    x = torch.randn(M, 1, d, device="cuda", generator=g).to(torch.bfloat16)
    out = torch.empty(M, 1, dtype=torch.float32, device="cuda")
    if M > 256:                                     # the 128-row-tile kernel: per-tile stamps of its first and last CTA
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        tl, ms, cy = [], [], []
        for i in range(max(args.steps, 3) + 3):
            torch.cuda.synchronize()
            e0.record()
            specdec.specdec_accept_head(ctx, x, Ws[i % copies], None, w_out, 0.1, out)
            e1.record()
            torch.cuda.synchronize()
            buf = (ctypes.c_longlong * 128)()
            lib.specdec_debug_head_tile_stamps(buf)
            raw = np.array(buf[:], dtype=np.float64).reshape(2, 8, 8)
            a = raw[:, :, :6]
            if i >= 3:
                tl.append(np.where(a > 0, (a - a[a > 0].min()) * 1e-3, np.nan))
                cy.append(np.where(raw[:, :, 3] > 0, raw[:, :, 7] - raw[:, :, 6], np.nan))   # main loop, SM cycles
                ms.append(e0.elapsed_time(e1))
        import warnings
        with warnings.catch_warnings():              # tiles a CTA does not have are NaN in every call
            warnings.simplefilter("ignore", RuntimeWarning)
            a = np.nanmedian(np.stack(tl), 0)
            cyc = np.nanmedian(np.stack(cy), 0)
        print(f"acceptance head, M={M} rows, d={d}, D={D}: tiles of the call's launch (all blocks: a CTA's tiles in the order it "
              f"works on them, first block first) on its first and its last CTA (a pair's MMA-side stamps are its even CTA's: "
              f"the last CTA of a paired launch has no row); microseconds from the launch's first stamp, median of {len(tl)} "
              f"isolated calls; whole call by CUDA events {1e3 * np.mean(ms):.1f} us")
        print("| CTA | tile | first k-block requested | accumulator free | first k-block landed | all MMAs issued | accumulator complete | epilogue done | main loop (landed to issued), SM cycles | SM MHz in it |\n|---|---|---|---|---|---|---|---|---|---|")
        f = lambda v: "-" if np.isnan(v) else f"{v:.2f}"
        for c in range(2):
            for t in range(8):
                if not np.isnan(a[c, t, 3]):
                    print(f"| {'first' if c == 0 else 'last'} | {t} | " + " | ".join(f(a[c, t, k]) for k in range(6))
                          + f" | {cyc[c, t]:.0f} | {cyc[c, t] / (a[c, t, 3] - a[c, t, 2]):.0f} |")
        ctx.close()
        return
    rows = []
    for i in range(max(args.steps, 3) + 3):
        torch.cuda.synchronize()
        specdec.specdec_accept_head(ctx, x, Ws[i % copies], None, w_out, 0.1, out)      # weights not seen for 5 calls: cold
        torch.cuda.synchronize()
        buf = (ctypes.c_longlong * 192)()
        lib.specdec_debug_head_stamps(buf)
        a = np.array(buf[:], dtype=np.float64).reshape(2, 6, 16)[:, :, :10]
        if i >= 3:
            rows.append(np.where(a > 0, (a - a[a > 0].min()) * 1e-3, np.nan))
    a = np.nanmedian(np.stack(rows), 0)
    names = ["CTA start", "barriers, tensor memory ready", "TMA: first weight tiles requested / MMA: first stage landed",
             "TMA: previous kernel complete, X requested / MMA: all MMAs issued", "epilogue warps: accumulator complete",
             "cluster barrier 1 (every ring consumed)", "lane quarters sent to their owners", "cluster barrier 2 (all partial sums in)",
             "epilogue done", "sigmoid by the last CTA (last block), CTA end"]
    print(f"acceptance head, M={M} rows, d={d}, D={D}, cold weights, one isolated call: one CTA of each of the two launches; "
          f"microseconds from the first CTA start, median of {len(rows)} calls")
    print("| phase | block 1: TMA warp | MMA warp | epilogue warp | block 2: TMA warp | MMA warp | epilogue warp |\n|---|---|---|---|---|---|---|")
    f = lambda v: "-" if np.isnan(v) else f"{v:.2f}"
    for k, nm in enumerate(names):
        print(f"| {nm} | {f(a[0, 0, k])} | {f(a[0, 1, k])} | {f(a[0, 2, k])} | {f(a[1, 0, k])} | {f(a[1, 1, k])} | {f(a[1, 2, k])} |")
    ctx.close()


def run_vocab_sharded(args, cfg):
    """One batch, its vocabulary split over the ranks: statistics -> all-gather -> accept tests and local
    masses -> all-gather -> draw -> max-reduction (strong scaling: the job is the same at every N)."""
    import torch.distributed as dist
    from paper_2405_19715_b200 import sharded, specdec
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    else:                                            # one rank still goes through the collectives
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(free_port()))
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    inp = wl.make_verify_inputs(cfg)                 # replicated: every rank draws the same job
    off, size = sharded.vocab_slices(cfg.V, world, multiple=8 if cfg.dtype == "bf16" else 4)[rank]
    ts = specdec.from_numpy(np.ascontiguousarray(inp["target_logits"][:, :, off:off + size])).to(dev)
    ds = specdec.from_numpy(np.ascontiguousarray(inp["draft_logits"][:, :, off:off + size])).to(dev)
    y = specdec.from_numpy(inp["cand_tokens"]).to(dev)
    L = specdec.from_numpy(inp["cand_len"]).to(dev)
    u = specdec.from_numpy(inp["uniforms"]).to(dev)
    ctx = specdec.Context(cfg.B, cfg.K)
    T = float(inp["temperature"])
    es = 2 if cfg.dtype == "bf16" else 4
    spoil = None if cfg.B * (2 * cfg.K + 1) * size * es > 2 * 126e6 else torch.zeros(64 << 20, dtype=torch.int32, device=dev)

    def step():
        if spoil is not None:
            spoil.sum()                              # reads 256 MB: the shard is out of L2 again
        return sharded.verify_correct_vocab_sharded(ctx, ts, ds, off, cfg.V, y, L, u, T)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    l0 = ctx.launch_count()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    dist.barrier()
    torch.cuda.synchronize()
    for a, b in evs:
        if spoil is not None:
            spoil.sum()
        a.record()
        n, tok = sharded.verify_correct_vocab_sharded(ctx, ts, ds, off, cfg.V, y, L, u, T)
        b.record()
    torch.cuda.synchronize()
    dist.barrier()
    ms = max_over_ranks(float(np.mean([a.elapsed_time(b) for a, b in evs])), world, dev)
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0:
        peaks = measured_peaks()
        tokens = float(inp["cand_len"].sum())
        alg_rank = algorithmic_bytes(cfg, inp["cand_len"], size)
        achieved = alg_rank / (ms * 1e-3) / 1e9
        line = {"metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": f"{cfg.name}: verify/correct with the vocabulary split over {world} rank(s) "
                                       f"({size} of {cfg.V} columns here), B={cfg.B} K={cfg.K} {cfg.dtype}; no head, no stop rule",
                           "sharding": f"vocabulary x{world}", "collectives": "2 all-gathers + 1 max-reduction (NCCL)",
                           "l2": "shard exceeds L2" if spoil is None else "256 MB read between steps"},
                "clocks": clocks, "gpu_launches": int(ctx.launch_count() - l0),
                "roofline": {"kernel": "sharded verify/correct (3 local phases + collectives), per rank", "bound": "hbm",
                             "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                             "peak_source": peaks["source"] + " copy bandwidth", "algorithmic_bytes": alg_rank,
                             "kernel_ms": ms, "traffic": None},
                "e2e": None}
        print(json.dumps(line), flush=True)
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
    ap.add_argument("--vocab-shards", action="store_true",
                    help="split the vocabulary of one batch over the ranks and time the sharded verify/correct")
    ap.add_argument("--sustained-seconds", type=float, default=2.0, help="length of the back-to-back loop (0 = skip)")
    ap.add_argument("--cpu-budget", type=float, default=10.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--early-exit", action="store_true",
                    help="run the timed step itself with SPECDEC_VERIFY_EARLY_EXIT (not the contract's path: positions "
                         "after a row's known first rejection are not read); the line says so in config")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the legs outside the timed region: warm figure, early exit, graph replay (profiling runs)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling runs)")
    ap.add_argument("--phases", action="store_true",
                    help="print per-phase device timestamps of the one-CTA-per-unit verify/correct kernel (diagnostic build)")
    ap.add_argument("--head-phases", action="store_true",
                    help="print phase timestamps of the weights-as-M head kernel for --batch rows (diagnostic build)")
    ap.add_argument("--stub-step", action="store_true", help="launcher self-check: gloo ranks on the CPU, empty step")
    args = ap.parse_args()
    if args.early_exit:
        args.kernel |= 0x100                          # SPECDEC_VERIFY_EARLY_EXIT
    cfg = wl.CONFIGS[args.workload]
    if args.batch:
        cfg = cfg.scaled(B=args.batch, name=f"{cfg.name}(B={args.batch})")
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:      # not under a launcher yet: start the ranks
        rc, out = launch_ranks(args.gpus, sys.argv[1:])
        for ln in out.splitlines():                            # the result line to stdout, NCCL's log to stderr
            print(ln, file=sys.stdout if ln.startswith("{") else sys.stderr, flush=True)
        sys.exit(rc)
    if args.stub_step:
        run_stub(args)
    elif args.head_phases:
        run_head_phases(args)
    elif args.phases:
        run_phases(args, cfg)
    elif args.vocab_shards:
        run_vocab_sharded(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
