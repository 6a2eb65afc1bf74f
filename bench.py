#!/usr/bin/env python
"""Benchmark of the DropMatch verification path: verify calls/s on the Llama-3-8B-shaped head.

One step = one whole verify call (Eq. 1 masks, Eq. 2-3 masked head, per-path argmax, token
counts, acceptance scan: at this size a 2 us mask pass and one launch of the fused kernel, whose
last CTA finishes the call) on one batch of synthetic input: d=4096, V=128256, bf16, T=5 draft
positions, K=8 dropout paths, p=0.1, B=1.
Prints ONE JSON line (rank 0).  `--gpus N` run as plain `python bench.py` starts N ranks itself
(one per GPU, independent replicas); under torchrun it joins the ranks it is given.
`--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "verify_calls_per_s"
UNIT = "calls/s"
WORKLOAD = "llama8b"   # Llama-3-8B-shaped head: the configuration the metric is quoted on

# DRAM bytes (read + write) of one fused head-kernel launch on this workload, from the ncu capture
# summarised in profiles/; None until a capture exists.
NCU_TRAFFIC_BYTES = {"llama8b": 1051385000 + 1604000, "llama8b_k32": 1052995000 + 1725000,
                     "llama8b_b2k32": 1080990000 + 2259000}


def load_peaks():
    path = ROOT / "MEASURED_PEAKS.json"
    if path.exists():
        p = json.loads(path.read_text())
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [x.strip() for x in line.split(",")]))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for (ts, r) in self.rows if (t0 is None or ts >= t0) and (t1 is None or ts <= t1 + 0.15)]
        rows = rows or [r for (_, r) in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def time_oracle(cfg, work_cpu, steps, warmup, budget_s=20.0):
    """Times the CPU oracle as it stands on whole verify calls; returns (calls/s, cores, sample, ms_per_step)."""
    import oracle
    from paper_2603_03333_b200 import workloads as wl
    Wn, Hn = wl.to_numpy_storage(work_cpu.W), wl.to_numpy_storage(work_cpu.H)
    draft = work_cpu.draft.numpy()
    # a bounded sample of the call: the first `pos` draft positions (K paths each) of sequence 0
    t0 = time.perf_counter()
    oracle.logits_row(Wn, cfg.dtype, Hn[0, 0], cfg.p, wl.MASK_SEED, 0, 0, 0)
    t_row = time.perf_counter() - t0
    rows_budget = max(1, int(budget_s / max(t_row, 1e-6) / max(1, steps + warmup)))
    pos = max(1, min(cfg.T, rows_budget // cfg.K))
    frac = pos / (cfg.B * cfg.T)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.verify_batched(Wn, cfg.dtype, Hn[:1, :pos], draft[:1, :pos], cfg.K, cfg.p, wl.MASK_SEED)
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    t_call = (sum(times) / len(times)) / frac      # scaled to the whole call (cost is linear in rows)
    sample = (f"{pos} of {cfg.B * cfg.T} draft positions x K={cfg.K} paths per step ({pos * cfg.K} of {cfg.rows} rows), "
              f"{len(times)} steps, scaled by rows")
    return 1.0 / t_call, oracle.threads(), sample, t_call * 1e3


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    """The slowest rank's figure (replicas run independently; the job is as slow as its slowest)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_calls_per_s(ms_total_local: float, steps: int, world: int, device="cpu"):
    """Whole-job throughput of `world` independent replicas that each ran `steps` verify calls:
    (world * steps) / (max over ranks of the timed region).  Returns (calls/s, ms per step)."""
    ms_total = max_over_ranks(ms_total_local, world, device)
    return world * steps / (ms_total * 1e-3), ms_total / steps


def parity_report(cfg, got_tokens, work_cpu):
    """One full comparison of a call's decoded tokens with the CPU oracle, outside every timed
    region: how many rows the oracle itself flags as near-ties (top-2 logit gap below 2e-2) and
    how many tokens differ (allowed only inside those rows)."""
    import oracle
    from paper_2603_03333_b200 import workloads as wl
    ref = oracle.verify_batched(wl.to_numpy_storage(work_cpu.W), cfg.dtype, wl.to_numpy_storage(work_cpu.H),
                                work_cpu.draft.numpy(), cfg.K, cfg.p, wl.MASK_SEED)
    differ = got_tokens != ref["tokens"]
    near = ref["gap"] < 2e-2
    return dict(rows_compared=int(differ.size), near_tie_rows=int(near.sum()), token_mismatches=int(differ.sum()),
                mismatches_outside_near_ties=int((differ & ~near).sum()), near_tie_gap=2e-2)


def self_launch(args) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script (one per GPU,
    rendezvous on 127.0.0.1) and pass rank 0's JSON line through."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(args.gpus):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")           # the communicator log (stderr) shows the rank count
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        procs.append(subprocess.Popen([sys.executable, str(Path(__file__).resolve()), *sys.argv[1:]], env=env,
                                      stdout=subprocess.PIPE if rank == 0 else subprocess.DEVNULL, text=True))
    out, _ = procs[0].communicate()
    rcs = [procs[0].returncode] + [p.wait() for p in procs[1:]]
    sys.stdout.write(out)
    sys.stdout.flush()
    return max(abs(rc) for rc in rcs)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2603_03333_b200 import workloads as wl
    cfg = wl.CONFIGS[WORKLOAD]
    work = wl.make_workload(cfg, device="cpu")
    steps, warmup = max(1, min(args.steps, 3)), max(0, min(args.warmup, 1))
    value, cores, sample, ms = time_oracle(cfg, work, steps, warmup, budget_s=60.0)
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=steps, warmup=warmup,
                ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic",
                config=dict(workload=WORKLOAD, d=cfg.d, V=cfg.V, B=cfg.B, T=cfg.T, K=cfg.K, p=cfg.p, rows=cfg.rows),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_2603_03333_b200 as pk
    from paper_2603_03333_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    backend = os.environ.get("DM_BENCH_BACKEND", "nccl")   # "gloo" + DM_BENCH_STUB: launcher test on CPU
    if os.environ.get("DM_BENCH_STUB"):
        return run_stub(args, rank, world, backend)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group(backend, device_id=torch.device(dev))

    cfg = wl.CONFIGS[args.workload]
    work = wl.make_workload(cfg, device=dev)       # every rank: an independent replica of the call
    ctx = pk.Context(local)
    ctx.set_head(work.W, max_rows=work.cfg.rows, max_hidden_rows=work.cfg.B * work.cfg.T)
    cfg = work.cfg                                 # a tree workload fixes its hidden-row count when drawn
    out = ctx.alloc_outputs(cfg.B, cfg.T, cfg.K) if cfg.kind == "chain" else None
    seed = wl.MASK_SEED

    def step(i):
        if cfg.kind == "chain":
            ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, seed + i, out=out)
        else:
            ctx.verify_tree(work.H, work.node_token, work.node_parent, work.node_hrow, cfg.K, cfg.p, seed + i)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin = time.perf_counter()
    ev0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    ev1.record()
    barrier()
    t_end = time.perf_counter()
    clocks = sampler.stop(t_begin, t_end)
    if ctx.device_error() != 0:
        raise SystemExit("device error word set during the timed region")
    ms_total = ev0.elapsed_time(ev1)
    launches_per_step = ctx.last_launches()
    impl_used = ctx.last_impl()
    value, ms_step = aggregate_calls_per_s(ms_total, args.steps, world, dev)

    # dominant kernel alone: events on the launching stream around the head kernel of each step
    ctx.profile_head(True)
    for i in range(min(args.steps, 200)):
        step(i)
    torch.cuda.synchronize()
    ms_sum, n_prof = ctx.profile_read()
    ctx.profile_head(False)
    head_ms_avg = ms_sum / max(1, n_prof)

    # read-only HBM ceiling of this machine, measured live: a plain streaming read of W (larger than L2)
    for _ in range(3):
        ctx.debug_read_stream(work.W)
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    for _ in range(20):
        ctx.debug_read_stream(work.W)
    r1.record()
    torch.cuda.synchronize()
    read_only_gbs = work.W.numel() * work.W.element_size() * 20 / (r0.elapsed_time(r1) * 1e-3) / 1e9

    elem = 2 if cfg.dtype == wl.BF16 else 4
    alg_bytes = (cfg.V * cfg.d + cfg.B * cfg.T * cfg.d) * elem
    alg_flops = 2.0 * cfg.rows * cfg.V * cfg.d
    peaks = load_peaks()
    t_mem, t_flop = alg_bytes / (peaks["hbm_gbs"] * 1e9), alg_flops / (peaks["bf16_tflops"] * 1e12)
    if t_mem >= t_flop:      # the bench workload: W streamed once per call bounds the kernel
        achieved = alg_bytes / (head_ms_avg * 1e-3) / 1e9
        roofline = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=achieved / peaks["hbm_gbs"], traffic=NCU_TRAFFIC_BYTES.get(args.workload),
                        peak_source=f"of {peaks['source']} (STREAM-style copy, burst)", algorithmic_bytes=alg_bytes)
    else:                    # many rows: the dense bf16 contraction bounds it
        achieved = alg_flops / (head_ms_avg * 1e-3) / 1e12
        roofline = dict(bound="tensor", achieved=achieved, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                        frac=achieved / peaks["bf16_tflops"], traffic=NCU_TRAFFIC_BYTES.get(args.workload),
                        peak_source=f"of {peaks['source']} (cuBLAS bf16, burst)", algorithmic_flops=alg_flops)
    roofline.update(kernel="fused_head_kernel", kernel_ms=head_ms_avg, read_only_stream_gbs=read_only_gbs,
                    frac_of_read_only_stream=(alg_bytes / (head_ms_avg * 1e-3) / 1e9) / read_only_gbs,
                    whole_call_gbs=alg_bytes / (ms_step * 1e-3) / 1e9)

    # end to end through the host-buffer entry point: H2D of H and draft, D2H of all results, per step
    e2e = None
    if cfg.kind == "chain":
        Hh, dh = work.H.cpu().pin_memory(), work.draft.cpu().pin_memory()
        hout = ctx.alloc_host_outputs(cfg.B, cfg.T, cfg.K)
        for i in range(max(args.warmup, 10)):   # untimed: first calls look up the pinned buffers and warm the host path
            ctx.verify_batched_host(Hh, dh, cfg.K, cfg.p, seed + i, out=hout)
        barrier()
        e0 = time.perf_counter()
        n_e2e = args.steps
        for i in range(n_e2e):
            ctx.verify_batched_host(Hh, dh, cfg.K, cfg.p, seed + i, out=hout)   # returns with the results on the host
        torch.cuda.synchronize()
        e_s = time.perf_counter() - e0
        e2e = dict(value=aggregate_calls_per_s(e_s * 1e3, n_e2e, world, dev)[0], unit=UNIT,
                   h2d_bytes_per_step=Hh.numel() * elem + dh.numel() * 4,
                   d2h_bytes_per_step=sum(v.numel() * 4 for v in hout.values()))

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16" if cfg.dtype == wl.BF16 else "f32", data="synthetic",
                config=dict(workload=args.workload, d=cfg.d, V=cfg.V, B=cfg.B, T=cfg.T, K=cfg.K, p=cfg.p,
                            rows=cfg.rows, l2="inputs larger than L2 (W is re-streamed from HBM every step)",
                            multi_gpu="replicas only: each rank verifies its own call, no collective",
                            impl={1: "simt", 2: "tcgen05"}.get(impl_used, "?")),
                clocks=clocks, e2e=e2e, gpu_launches=launches_per_step * args.steps, roofline=roofline)

    if rank == 0 and world == 1 and not args.no_cpu_baseline and cfg.kind == "chain":
        work_cpu = wl.Workload(cfg, work.W.cpu(), work.H.cpu(), work.draft.cpu(), None, None, None)
        v, cores, sample, _ = time_oracle(cfg, work_cpu, steps=1, warmup=0, budget_s=15.0)
        line["cpu_baseline"] = dict(value=v, unit=UNIT, cores=cores, kind="oracle", sample=sample)
        if cfg.rows <= 64:     # the whole call through the oracle once more: seconds at this size
            got = ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED, out=out)
            torch.cuda.synchronize()
            line["parity"] = parity_report(cfg, got["tokens"].cpu().numpy(), work_cpu)
    if rank == 0:
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_stub(args, rank, world, backend):
    """Launcher check without a GPU: every rank 'times' a fixed duration and the ranks aggregate
    exactly as the real run does; rank 0 prints a line with the rank count."""
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group(backend)
    value, ms_step = aggregate_calls_per_s(100.0 * (rank + 1), args.steps, world)
    if rank == 0:
        print(json.dumps(dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
                              ms_per_step=ms_step, stub=True)), flush=True)
    if world > 1:
        dist.destroy_process_group()


SWEEPS = {
    # (head name, V, d, [(B, T, K), ...]): call sizes from 8 paths to the tensor-bound range
    "llama8b": (128256, 4096, [(1, 1, 8), (1, 2, 8), (1, 5, 8), (1, 8, 8), (1, 5, 16), (1, 8, 16), (1, 5, 32),
                               (1, 7, 32), (1, 8, 32), (3, 5, 20), (4, 8, 16), (8, 8, 16)]),
    "qwen8b": (151936, 4096, [(B, 7, K) for B in (1, 8, 32) for K in (4, 8, 16, 32)]),
    "llama70b": (128256, 8192, [(1, 8, 16), (16, 8, 16)]),
}


def run_sweep(args):
    """Not the benchmark line: times the head kernel(s) and the whole call over a list of call
    sizes on one head and prints one JSON line per size (fractions against the measured peaks)."""
    import torch
    import paper_2603_03333_b200 as pk
    from paper_2603_03333_b200 import workloads as wl
    V, d, cases = SWEEPS[args.sweep]
    dev, peaks = "cuda:0", load_peaks()
    W = wl.make_head(V, d, wl.BF16, seed=1, device=dev)
    ctx = pk.Context(0)
    ctx.set_head(W, max_rows=max(B * T * K for B, T, K in cases), max_hidden_rows=max(B * T for B, T, K in cases))
    for B, T, K in cases:
        H = wl.make_hidden(B * T, d, wl.BF16, seed=2, device=dev).view(B, T, d)
        draft = torch.zeros((B, T), dtype=torch.int32, device=dev)
        out = ctx.alloc_outputs(B, T, K)
        rows, reps = B * T * K, (50 if B * T * K <= 512 else 8)
        for i in range(5):
            ctx.verify_batched(H, draft, K, 0.1, 1 + i, out=out)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            ctx.verify_batched(H, draft, K, 0.1, 100 + i, out=out)
        e1.record()
        torch.cuda.synchronize()
        ctx.profile_head(True)
        for i in range(reps):
            ctx.verify_batched(H, draft, K, 0.1, 100 + i, out=out)
        torch.cuda.synchronize()
        ms, n = ctx.profile_read()
        ctx.profile_head(False)
        t_head, t_call = ms / n * 1e-3, e0.elapsed_time(e1) / reps * 1e-3
        t_mem = (V * d + B * T * d) * 2 / (peaks["hbm_gbs"] * 1e9)
        t_flop = 2.0 * rows * V * d / (peaks["bf16_tflops"] * 1e12)
        print(json.dumps(dict(head=args.sweep, B=B, T=T, K=K, rows=rows, head_us=round(t_head * 1e6, 1),
                              call_us=round(t_call * 1e6, 1), bound="hbm" if t_mem >= t_flop else "tensor",
                              frac=round(max(t_mem, t_flop) / t_head, 3), launches=ctx.last_launches())), flush=True)
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", default=None, choices=sorted(SWEEPS), help="time a list of call sizes on one head")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.sweep:
        if args.impl == "reference":
            os.environ.update(RANK="0", WORLD_SIZE=str(args.gpus))     # rank 0 alone runs the oracle
        else:
            raise SystemExit(self_launch(args))
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
