#!/usr/bin/env python
"""Benchmark of the FP8 block-scaled MoE forward on B200 (one JSON line on stdout).

A "step" is one pass of the whole hot path over one synthetic batch of the training-forward
MoE shape (M = 32768 tokens of hidden 2048, 128 experts, top-8, Zipf(1.1) popularity):
on-the-fly weight quantization of the layer's bf16 masters (w13, w2), then the routed MoE FFN
(quantize activations, group by expert, gate_up grouped GEMM + SwiGLU + re-quantization, down
grouped GEMM + weighting, fixed-order combine).  The decode shape (M = 256, weights already
quantized, as in the rollout engine) is measured in the same run and reported under "decode".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--dry-run]

N > 1 runs one rank per GPU: data-parallel replicas over independent token batches, weights
replicated, no collective on the data path (weak scaling).  Started under torch.distributed.run the
script takes its rank from the environment; started plainly with --gpus N > 1 it starts the N ranks
itself (it re-executes under torch.distributed.run on 127.0.0.1).  --dry-run only brings the ranks up
(NCCL, or gloo without a GPU), gathers their ranks and prints the world size.
--impl reference times the CPU oracle (test infrastructure) on the host cores on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

H, I, E, TOPK = 2048, 768, 128, 8
M_TRAIN, M_DECODE = 32768, 256
FLOP_PER_TOKEN = TOPK * 2 * (H * 2 * I + I * H)          # 75.5 MFLOP
METRIC = "FP8 MoE-layer tokens/s"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024


def peaks():
    """Measured roofline denominators (generated file), else the documented fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(source="measured", hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])))
    return dict(source="fallback", hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0)


# --------------------------------------------------------------------------- inputs (device)
def make_inputs(m: int, seed: int, device, zipf: bool):
    """Synthetic layer of Qwen3-30B-A3B FFN shape, generated on the device: W ~ N(0, 0.02^2),
    X ~ N(0, 1) with 1% of entries x50, router logits ~ N(0, 1) (+ ln Zipf(1.1) popularity for
    the training shape), top-8 with softmax weights over the selected logits."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    w13 = (torch.randn((E, 2 * I, H), generator=g, device=device) * 0.02).to(torch.bfloat16)
    w2 = (torch.randn((E, H, I), generator=g, device=device) * 0.02).to(torch.bfloat16)
    x = torch.randn((m, H), generator=g, device=device)
    x = torch.where(torch.rand((m, H), generator=g, device=device) < 0.01, x * 50.0, x).to(torch.bfloat16)
    logits = torch.randn((m, E), generator=g, device=device, dtype=torch.float64)
    if zipf:
        rank = torch.randperm(E, generator=g, device=device).to(torch.float64) + 1.0
        p = rank ** -1.1
        logits = logits + torch.log(p / p.sum())[None, :]
    sel, ids = torch.topk(logits, TOPK, dim=1)
    wts = torch.softmax(sel, dim=1).to(torch.float32)
    return w13, w2, x, ids.to(torch.int32).contiguous(), wts.contiguous()


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self, gpu_index: int) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        self.p.wait()
        self.f.flush()
        sm, smax, reasons, power = [], [], set(), []
        for line in open(self.f.name):
            c = [t.strip() for t in line.split(",")]
            if len(c) < 9 or not c[0].isdigit() or int(c[0]) != gpu_index:
                continue
            try:
                sm.append(float(c[1])); smax.append(float(c[2])); power.append(float(c[3]))
            except ValueError:
                continue
            for name, v in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.f.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [s for s, w in zip(sm, power) if w > 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# --------------------------------------------------------------------------- CPU oracle arm
def cpu_reference_step(state, n_tokens, n_experts_q):
    """One bounded oracle step; returns the estimated seconds of a full step (scaled linearly
    in experts for the quantization part and in tokens for the layer part)."""
    import oracle
    t0 = time.perf_counter()
    oracle.quantize_weight(state["w13"][:n_experts_q])
    oracle.quantize_weight(state["w2"][:n_experts_q])
    t_q = time.perf_counter() - t0
    t0 = time.perf_counter()
    state["out"] = oracle.moe(state["x"][:n_tokens], state["ids"][:n_tokens], state["wts"][:n_tokens],
                              state["w13c"], state["w13s"], state["w2c"], state["w2s"])
    t_m = time.perf_counter() - t0
    return t_q * (E / n_experts_q) + t_m * (M_TRAIN / n_tokens), t_q + t_m


def cpu_state(seed: int, n_tokens: int):
    """Host copies of a synthetic layer for the oracle (same recipe, host RNG), with the
    weights quantized by the oracle (untimed set-up)."""
    import oracle
    from paper_2604_07853_b200 import inputs
    rng = np.random.default_rng(seed)
    w13 = inputs.weight_bf16(rng, E, 2 * I, H)
    w2 = inputs.weight_bf16(rng, E, H, I)
    x = inputs.act_bf16(rng, n_tokens, H)
    ids, wts = inputs.routing(rng, n_tokens, E, TOPK, inputs.zipf_log_popularity(rng, E, 1.1))
    w13c, w13s = oracle.quantize_weight(w13)
    w2c, w2s = oracle.quantize_weight(w2)
    return dict(w13=w13, w2=w2, x=x, ids=ids, wts=wts, w13c=w13c, w13s=w13s, w2c=w2c, w2s=w2s)


def run_reference(args, rank: int):
    """--impl reference: the CPU oracle as it stands, on the host cores, bounded sample."""
    if rank != 0:
        return
    import oracle
    n_tokens, n_exp = 512, 8      # per step: about a second of oracle work on 8-16 cores
    st = cpu_state(4, n_tokens)
    for _ in range(args.warmup):
        cpu_reference_step(st, n_tokens, n_exp)
    est, raw = [], []
    for _ in range(args.steps):
        e, r = cpu_reference_step(st, n_tokens, n_exp)
        est.append(e); raw.append(r)
    full_step_s = sum(est) / len(est)
    value = M_TRAIN / full_step_s
    cores = oracle.num_threads()
    sample = (f"per step: oracle quantize_weight on {n_exp} of {E} experts (scaled x{E // n_exp}) + "
              f"oracle MoE layer on {n_tokens} of {M_TRAIN} tokens (scaled x{M_TRAIN // n_tokens})")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup,
        # what was timed: one bounded sample step; the whole-step figure behind `value` is the
        # linear extrapolation named in `sample`
        "ms_per_step": sum(raw) / len(raw) * 1e3, "extrapolated_full_step_ms": full_step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3",
        "data": "synthetic", "config": config_dict(world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "note": "rank 0 alone runs the oracle; it uses no GPU",
    }))


def config_dict(n_gpus: int) -> dict:
    return {"workload": f"moe_ffn_train_fwd_M{M_TRAIN}_zipf1.1 (+ on-the-fly weight quantization)",
            "tokens_per_gpu": M_TRAIN, "hidden": H, "intermediate": I, "experts": E, "top_k": TOPK,
            "format": "fp8 e4m3, 128x128 weight blocks, 1x128 activation groups, fp32 scales",
            "l2": "inputs larger than L2 (1.2 GB bf16 masters + 0.6 GB codes + 0.13 GB activations per step)",
            "parallelism": f"dp{n_gpus} replicas, no collective"}


def spawn_ranks(n: int) -> int:
    """Started without a launcher but asked for n > 1 GPUs: run the same command line as n ranks of one
    node under torch.distributed.run (rendezvous on 127.0.0.1) and return its exit code."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def dry_run(rank: int, local_rank: int, world: int):
    """Bring the ranks up and let rank 0 print who is there: checks the launch path without timing
    anything (NCCL on GPUs, gloo on a CPU-only box)."""
    import torch.distributed as dist
    backend = "nccl" if torch.cuda.is_available() else "gloo"
    ranks = [0]
    if world > 1:
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
            t = torch.tensor([rank], device=torch.device("cuda", local_rank))
        else:
            dist.init_process_group("gloo")
            t = torch.tensor([rank])
        got = [torch.zeros_like(t) for _ in range(world)]
        dist.all_gather(got, t)
        ranks = sorted(int(g.item()) for g in got)
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"dry_run": True, "metric": METRIC, "n_gpus": world, "ranks": ranks, "backend": backend,
                          "scaling": "weak", "config": config_dict(world)}))


def source_hash() -> str:
    """Hash of the sources the dominant kernel is built from (ties a stored ncu figure to the code)."""
    h = hashlib.sha256()
    for f in ("gemm_sm100.cu", "ptx_sm100.cuh", "common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2604_07853_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def stored_traffic(tokens: int):
    """DRAM bytes per launch of the gate_up GEMM from the committed ncu summary, or None when the
    summary was taken from other sources than the ones in the tree (stale) or for another size."""
    path = os.path.join(ROOT, "profiles", "gemm_blockscaled_gate_up__dram_traffic.txt")
    if not os.path.exists(path):
        return None
    kv = dict(re.findall(r"^([a-z_0-9]+):\s*(\S+)", open(path).read(), flags=re.M))
    if kv.get("source_sha256_16") != source_hash() or int(kv.get("tokens", "0")) != tokens:
        return None
    return int(kv["dram_bytes_per_launch"])


# --------------------------------------------------------------------------- GPU arm
def main():
    global M_TRAIN
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=0, help="steps of the end-to-end region (0: --steps, at least 4, at most 100)")
    ap.add_argument("--no-peaks", action="store_true", help="skip the FP8-MMA and read-stream peak kernels (profiler captures)")
    ap.add_argument("--no-w4a16", action="store_true")
    ap.add_argument("--no-ep", action="store_true", help="skip the expert-parallel form of the layer")
    ap.add_argument("--ep", action="store_true",
                    help="with --gpus N > 1: split the experts across the ranks (two NCCL all-to-alls per layer) "
                         "in the expert_parallel section instead of running it as one rank per GPU")
    ap.add_argument("--no-backward", action="store_true")
    ap.add_argument("--no-tbpo", action="store_true")
    ap.add_argument("--no-router", action="store_true")
    ap.add_argument("--no-linear", action="store_true")
    ap.add_argument("--dry-run", action="store_true", help="start the ranks, print the world size, time nothing")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="length of the second (per-step timed) region used for mean / median / min")
    ap.add_argument("--tokens", type=int, default=M_TRAIN,
                    help="tokens per GPU of the training-shape step (smaller values are for profiler captures "
                         "only; the reported config names the size)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    M_TRAIN = args.tokens
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")

    if args.dry_run:
        dry_run(rank, local_rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch.distributed as dist
    from paper_2604_07853_b200 import binding, build, sharding

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if local_rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    ctx = binding.Context(local_rank)
    pk = peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v: float) -> float:
        return sharding.max_over_ranks(v, dev)

    # ---------------- training-forward shape: the headline step
    w13, w2, x, ids, wts = make_inputs(M_TRAIN, 1000 + rank, dev, zipf=True)
    w13c = torch.empty(w13.shape, dtype=torch.uint8, device=dev)
    w13s = torch.empty((E, 2 * I // 128, H // 128), dtype=torch.float32, device=dev)
    w2c = torch.empty(w2.shape, dtype=torch.uint8, device=dev)
    w2s = torch.empty((E, H // 128, I // 128), dtype=torch.float32, device=dev)
    out = torch.empty((M_TRAIN, H), dtype=torch.bfloat16, device=dev)
    ws = torch.empty(ctx.moe_workspace_bytes(M_TRAIN, H, I, E, TOPK), dtype=torch.uint8, device=dev)

    def step(xd=x, idd=ids, wtd=wts):
        ctx.quantize_weight(w13, w13c, w13s)
        ctx.quantize_weight(w2, w2c, w2s)
        ctx.moe_fwd(xd, idd, wtd, w13c, w13s, w2c, w2s, out=out, workspace=ws)

    sampler = ClockSampler()
    if rank == 0:
        sampler.start()          # nvidia-smi needs a moment to start: begin before the warm-up
    for _ in range(args.warmup):
        step()
    ctx.check_device_status()
    barrier()
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1))
    launches = ctx.launch_count() - launches0
    ctx.check_device_status()
    ms_step = ms_total / args.steps
    value = world * M_TRAIN / (ms_step * 1e-3)

    # A second region of at least --min-seconds, every step bracketed by its own events: mean, median
    # and min per step, at the clocks the part settles to under a seconds-long load.
    n_long = int(min(max(args.steps, args.min_seconds * 1e3 / ms_step * 1.05), 20000))
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_long + 1)]
    barrier()
    evs[0].record()
    for i in range(n_long):
        step()
        evs[i + 1].record()
    barrier()
    per_step = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_long)]
    long_ms = evs[0].elapsed_time(evs[n_long])
    timing = {"region_steps": n_long, "region_s": long_ms * 1e-3, "mean_ms": max_over_ranks(long_ms / n_long),
              "median_ms": max_over_ranks(statistics.median(per_step)), "min_ms": max_over_ranks(min(per_step)),
              "first_region_s": ms_total * 1e-3}
    del evs

    # A third region of the same length with every kernel bracketed by events (stage timing): the
    # per-kernel durations the roofline uses.  Headline and stage times are separate measurements.
    ctx.profile_begin(max_marks=n_long * 16 + 8)
    for _ in range(n_long):
        step()
    barrier()
    stages = ctx.profile_end()
    clocks = sampler.stop(local_rank) if rank == 0 else None
    ctx.check_device_status()

    # ---------------- the build's own roofline denominators (harness kernels, same run)
    own = {}
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, kb, reps in (() if args.no_peaks else (("burst", 30000, 5), ("sustained", 300000, 10))):
        best, total_ms, fl = None, 0.0, 0.0
        for _ in range(reps):
            ev2.record()
            fl = ctx.harness_fp8_mma_peak(kb)
            ev3.record()
            torch.cuda.synchronize()
            t = ev2.elapsed_time(ev3)
            total_ms += t
            best = t if best is None else min(best, t)
        own[f"fp8_mma_tflops_{name}"] = fl / ((best if name == "burst" else total_ms / reps) * 1e-3) / 1e12
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    best = None
    for _ in range(0 if args.no_peaks else 5):
        ev2.record()
        ctx.harness_read_stream(w13, sink)
        ev3.record()
        torch.cuda.synchronize()
        t = ev2.elapsed_time(ev3)
        best = t if best is None else min(best, t)
    own["read_gbs"] = w13.numel() * 2 / (best * 1e-3) / 1e9 if best else None
    own["note"] = ("fp8_mma: one thread per SM issuing tcgen05.mma kind::f8f6f4 128x256x32 on operands resident in "
                   "shared memory (burst: best of 5 launches of ~10 ms; sustained: mean of 10 launches of ~0.1 s); "
                   "read: 16-byte loads over the 1.2 GB of bf16 masters, best of 5")
    ctx.check_device_status()

    # realised group sizes of the Zipf(1.1) routing (rows per expert), and how full the 128-row tiles are
    rows_e = torch.bincount(ids.flatten().to(torch.int64), minlength=E).cpu().numpy()
    tiles_e = (rows_e + 127) // 128
    group_hist = {"min": int(rows_e.min()), "median": float(np.median(rows_e)), "max": int(rows_e.max()),
                  "empty_experts": int((rows_e == 0).sum()), "row_tiles": int(tiles_e.sum()),
                  "tile_fill": float(rows_e.sum() / max(1, tiles_e.sum() * 128))}

    # ---------------- end to end: pinned host inputs in, result out, copies inside the timing
    # Three streams (copy in / compute / copy out) with double-buffered device and host buffers, as a
    # trainer's input pipeline would run it: step i's inputs cross PCIe while step i-1 computes and
    # step i-2's result goes back.  Every step's copies are inside the timed region.
    hx, hids, hwts = x.cpu().pin_memory(), ids.cpu().pin_memory(), wts.cpu().pin_memory()
    houts = [torch.empty((M_TRAIN, H), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    dins = [(torch.empty_like(x), torch.empty_like(ids), torch.empty_like(wts)) for _ in range(2)]
    douts = [torch.empty_like(out) for _ in range(2)]
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def e2e_run(n):
        in_done, cmp_done, out_done = [], [], []
        for i in range(n):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(cmp_done[i - 2])        # the device input buffer is free again
                dins[b][0].copy_(hx, non_blocking=True)
                dins[b][1].copy_(hids, non_blocking=True)
                dins[b][2].copy_(hwts, non_blocking=True)
                e = torch.cuda.Event()
                e.record(s_in)
                in_done.append(e)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(in_done[i])
                if i >= 2:
                    s_cmp.wait_event(out_done[i - 2])       # the device output buffer is free again
                ctx.quantize_weight(w13, w13c, w13s)
                ctx.quantize_weight(w2, w2c, w2s)
                ctx.moe_fwd(*dins[b], w13c, w13s, w2c, w2s, out=douts[b], workspace=ws)
                e = torch.cuda.Event()
                e.record(s_cmp)
                cmp_done.append(e)
            with torch.cuda.stream(s_out):
                s_out.wait_event(cmp_done[i])
                houts[b].copy_(douts[b], non_blocking=True)
                e = torch.cuda.Event()
                e.record(s_out)
                out_done.append(e)
        return out_done

    e2e_steps = 0 if args.no_e2e else (args.e2e_steps if args.e2e_steps > 0 else max(4, min(args.steps, 100)))
    if e2e_steps:
        e2e_run(4)
    barrier()
    cur = torch.cuda.current_stream()
    ev0.record()
    if e2e_steps:
        for st_ in (s_in, s_cmp, s_out):
            st_.wait_event(ev0)
        for e in e2e_run(e2e_steps)[-2:]:
            cur.wait_event(e)                               # the last results are on the host
        cur.wait_stream(s_cmp)
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1)) / max(e2e_steps, 1) if e2e_steps else None
    ctx.check_device_status()
    e2e = {"value": world * M_TRAIN / (e2e_ms * 1e-3) if e2e_ms else None, "unit": UNIT, "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": hx.numel() * 2 + hids.numel() * 4 + hwts.numel() * 4,
           "d2h_bytes_per_step": houts[0].numel() * 2,
           "note": "bf16 masters stay resident on the device; activations and routing in, layer output out, every "
                   "step, from/to pinned host memory; copy-in, compute and copy-out on three streams, double-buffered; "
                   "the region includes the pipeline's fill and drain (one copy-in and one copy-out that overlap nothing)",
           "steps": e2e_steps}
    del dins, douts

    # ---------------- roofline of the dominant kernel (gate_up grouped GEMM, tensor-bound)
    gu_ms, gu_n = stages["gate_up_gemm"]
    gu_ms_avg = gu_ms / max(gu_n, 1)
    gu_flops = M_TRAIN * TOPK * 2.0 * H * 2 * I                     # algorithmic flops per launch
    achieved = gu_flops / (gu_ms_avg * 1e-3) / 1e12
    # The kernel was timed inside a region of >= 2 s, so the sustained figure is its denominator
    # (fp8 = 2 x bf16, the nominal ratio); the other denominators are printed beside it.
    long_region = timing["region_s"] >= 1.0
    peak = 2.0 * (pk["bf16_sustained"] if long_region else pk["bf16_burst"])
    roofline = {"kernel": "gemm_blockscaled_kernel<gate_up>", "bound": "tensor", "achieved": achieved,
                "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": f"2 x bf16 {'sustained' if long_region else 'burst'} of {pk['source']} "
                               f"(kernel timed inside a {timing['region_s']:.1f} s region)",
                "frac_of_2x_bf16_burst": achieved / (2.0 * pk["bf16_burst"]),
                "frac_of_2x_bf16_sustained": achieved / (2.0 * pk["bf16_sustained"]),
                "frac_of_nominal_4500": achieved / 4500.0,
                "peak_fp8_measured": own.get("fp8_mma_tflops_sustained"), "peak_fp8_measured_burst": own.get("fp8_mma_tflops_burst"),
                "frac_of_own_fp8_mma_sustained": achieved / own["fp8_mma_tflops_sustained"] if "fp8_mma_tflops_sustained" in own else None,
                "peak_read_gbs": own["read_gbs"],
                # dram__bytes_read + write of one launch, from the committed ncu summary if it was
                # taken from the sources in the tree at this size; else null
                "traffic": stored_traffic(M_TRAIN), "source_sha256_16": source_hash(),
                "ms_per_launch": gu_ms_avg,
                "down_gemm": {"ms_per_launch": stages["down_gemm"][0] / max(stages["down_gemm"][1], 1),
                              "tflops": M_TRAIN * TOPK * 2.0 * I * H / (stages["down_gemm"][0] / max(stages["down_gemm"][1], 1) * 1e-3) / 1e12}}
    stage_ms = {k: (v[0] / max(n_long, 1)) for k, v in stages.items()}
    qw_ms = stage_ms.get("quantize_weight", 0.0)
    quant_weight = {"ms_per_step": qw_ms, "algorithmic_bytes": 3 * (w13.numel() + w2.numel()),
                    "gbs": 3 * (w13.numel() + w2.numel()) / (qw_ms * 1e-3) / 1e9 if qw_ms else None,
                    "frac_hbm_measured": 3 * (w13.numel() + w2.numel()) / (qw_ms * 1e-3) / 1e9 / pk["hbm_gbs"] if qw_ms else None}
    layer_ms = sum(stage_ms[k] for k in ("permute", "quantize_act", "gate_up_gemm", "down_gemm", "combine"))

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp8_e4m3", "data": "synthetic", "config": config_dict(world),
        "tflops": value * FLOP_PER_TOKEN / 1e12, "timing": timing, "stage_ms_per_step": stage_ms,
        "group_sizes": group_hist, "quantize_weight": quant_weight, "own_peaks": own,
        "moe_layer_only": {"ms": layer_ms, "tokens_per_s": M_TRAIN / (layer_ms * 1e-3),
                           "tflops": M_TRAIN * FLOP_PER_TOKEN / (layer_ms * 1e-3) / 1e12,
                           "frac_fp8_peak_measured": M_TRAIN * FLOP_PER_TOKEN / (layer_ms * 1e-3) / 1e12 / peak,
                           "frac_fp8_peak_nominal_4500": M_TRAIN * FLOP_PER_TOKEN / (layer_ms * 1e-3) / 1e12 / 4500.0},
        "roofline": roofline, "e2e": e2e, "gpu_launches": launches * world, "clocks": clocks,
    }

    # ---------------- dense projection (QKV of the training configuration): N = 5120, K = 2048, M = 8192 and 64
    if not args.no_linear:
        Nl, Kl = 5120, 2048
        gen = torch.Generator(device=dev).manual_seed(6000 + rank)
        wl = (torch.randn((Nl, Kl), generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
        # 16 copies of the quantized weight (168 MB), used in turn: a small-M call never finds its weight in L2
        copies = [ctx.quantize_weight(wl) for _ in range(16)]
        lin = {}
        for Ml in (8192, 64):
            xl = torch.randn((Ml, Kl), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
            yl = torch.empty((Ml, Nl), dtype=torch.bfloat16, device=dev)
            lsteps = max(args.steps, 20) * (1 if Ml > 1000 else 5)
            for i in range(5):
                ctx.linear_fwd(xl, *copies[i % 16], out=yl)
            barrier()
            ev0.record()
            for i in range(lsteps):
                ctx.linear_fwd(xl, *copies[i % 16], out=yl)
            ev1.record()
            barrier()
            l_ms = max_over_ranks(ev0.elapsed_time(ev1)) / lsteps
            ctx.profile_begin(max_marks=lsteps * 4 + 8)
            for i in range(lsteps):
                ctx.linear_fwd(xl, *copies[i % 16], out=yl)
            lst = ctx.profile_end()
            ctx.check_device_status()
            g_ms = lst["linear_gemm"][0] / max(lst["linear_gemm"][1], 1)
            fl = 2.0 * Ml * Nl * Kl
            lbytes = Nl * Kl + Nl * Kl // (128 * 128) * 4 + Ml * Kl * 2 + Ml * Nl * 2
            lin[f"M{Ml}"] = {
                "ms_per_call": l_ms, "gemm_ms": g_ms, "quantize_act_ms": lst["quantize_act"][0] / max(lst["quantize_act"][1], 1),
                "gemm_tflops": fl / (g_ms * 1e-3) / 1e12,
                "gemm_frac_fp8_peak_measured": fl / (g_ms * 1e-3) / 1e12 / (2.0 * pk["bf16_sustained"]),
                "algorithmic_bytes": lbytes, "gbs": lbytes / (l_ms * 1e-3) / 1e9,
                "frac_hbm_measured": lbytes / (l_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
            }
            del xl, yl
        result["linear"] = {"workload": f"dense FP8 projection N={Nl} K={Kl} (activation quantization + GEMM), "
                                        "16 weight copies used in turn", **lin}
        del wl, copies

    # ---------------- router (bf16 logits GEMM + top-k softmax) on the training batch
    if not args.no_router:
        gen = torch.Generator(device=dev).manual_seed(5000 + rank)
        wr = (torch.randn((E, H), generator=gen, device=dev, dtype=torch.float32) * 0.05).to(torch.bfloat16)
        rsteps = max(args.steps, 20)
        for _ in range(3):
            ctx.router_fwd(x, wr, TOPK)
        barrier()
        ev0.record()
        for _ in range(rsteps):
            ctx.router_fwd(x, wr, TOPK)
        ev1.record()
        barrier()
        r_ms = max_over_ranks(ev0.elapsed_time(ev1)) / rsteps
        ctx.check_device_status()
        rbytes = M_TRAIN * H * 2 + E * H * 2 + 2 * M_TRAIN * E * 4 + M_TRAIN * TOPK * 8
        result["router"] = {
            "workload": f"router forward, M={M_TRAIN} H={H} E={E} top-{TOPK} (bf16 logits GEMM with the top-k softmax in its epilogue, 1 launch)",
            "ms_per_step": r_ms, "tokens_per_s": world * M_TRAIN / (r_ms * 1e-3),
            "algorithmic_bytes": rbytes, "gbs": rbytes / (r_ms * 1e-3) / 1e9,
            "frac_hbm_measured": rbytes / (r_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
        }
        del wr

    # ---------------- expert-parallel form of the layer: dispatch / experts / combine as separate calls, the
    # rows exchanged between them (nothing to exchange with one rank; --ep splits the experts over the ranks)
    if not args.no_ep:
        from paper_2604_07853_b200.expert_parallel import CudaStages, ExpertParallelMoE, expert_range, run_local
        ep_world = world if (args.ep and world > 1) else 1
        ep_rank = rank if ep_world > 1 else 0
        lo, hi = expert_range(ep_rank, ep_world, E)
        ep = ExpertParallelMoE(CudaStages(ctx, (w13c[lo:hi], w13s[lo:hi]), (w2c[lo:hi], w2s[lo:hi]), E),
                               ep_rank, ep_world, E)

        def ep_fwd():
            return ep.forward(x, ids, wts) if ep_world > 1 else run_local([ep], [(x, ids, wts)])[0]

        same = None
        if ep_world == 1:
            ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, out=out, workspace=ws)
            same = bool(torch.equal(ep_fwd(), out))
        esteps = max(args.steps // 4, 10)
        for _ in range(3):
            ep_fwd()
        barrier()
        ev0.record()
        for _ in range(esteps):
            ep_fwd()
        ev1.record()
        barrier()
        ep_ms = max_over_ranks(ev0.elapsed_time(ev1)) / esteps
        ctx.check_device_status()
        result["expert_parallel"] = {
            "workload": f"moe_ffn_train_M{M_TRAIN} layer forward as dispatch / experts / combine stages, "
                        f"{ep_world} expert-parallel rank(s)"
                        + (" with NCCL all-to-all exchanges" if ep_world > 1 else " (no exchange; one host sync per layer for the row counts)"),
            "ms_per_layer": ep_ms, "tokens_per_s": world * M_TRAIN / (ep_ms * 1e-3),
            "bytewise_equal_to_fused_layer": same,
        }
        del ep

    # ---------------- 4-bit weight-only variants of the same layer (bf16 activations): integer codes with a
    # zero point ("w4a16") and e2m1 floating point ("fp4a16"); same storage, same kernels
    def bench_4bit(label, quantize, moe_fwd):
        q13 = quantize(w13)
        q2 = quantize(w2)
        ws4 = torch.empty(ctx.moe_w4a16_workspace_bytes(M_TRAIN, H, I, E, TOPK), dtype=torch.uint8, device=dev)

        def step4():
            quantize(w13, out=q13)
            quantize(w2, out=q2)
            moe_fwd(x, ids, wts, q13, q2, out=out, workspace=ws4)

        steps4 = max(args.steps // 2, 10)
        for _ in range(3):
            step4()
        barrier()
        ev0.record()
        for _ in range(steps4):
            step4()
        ev1.record()
        barrier()
        ms4 = max_over_ranks(ev0.elapsed_time(ev1)) / steps4
        ctx.profile_begin(max_marks=steps4 * 16 + 8)
        for _ in range(steps4):
            step4()
        st4 = ctx.profile_end()
        ctx.check_device_status()
        gu4 = st4["gate_up_gemm"][0] / max(st4["gate_up_gemm"][1], 1)
        dn4 = st4["down_gemm"][0] / max(st4["down_gemm"][1], 1)
        gu_tf = 2.0 * M_TRAIN * TOPK * H * 2 * I / (gu4 * 1e-3) / 1e12
        dn_tf = 2.0 * M_TRAIN * TOPK * I * H / (dn4 * 1e-3) / 1e12
        w4 = {
            "workload": f"moe_ffn_train_M{M_TRAIN} with {label} weights (per-step 4-bit quantization + layer forward)",
            "ms_per_step": ms4, "tokens_per_s": world * M_TRAIN / (ms4 * 1e-3),
            "stage_ms": {k: v[0] / steps4 for k, v in st4.items() if v[1]},
            "gate_up_tflops": gu_tf, "down_tflops": dn_tf,
            "gate_up_frac_bf16_peak_measured_sustained": gu_tf / pk["bf16_sustained"],
            "gate_up_frac_bf16_peak_measured_burst": gu_tf / pk["bf16_burst"],
        }
        # decode shape on pre-quantized weights; two weight copies alternated so that no step
        # re-reads a copy that is resident in L2
        _, _, xd4, idd4, wtd4 = make_inputs(M_DECODE, 2000 + rank, dev, zipf=False)
        outd4 = torch.empty((M_DECODE, H), dtype=torch.bfloat16, device=dev)
        sets4 = [(q13, q2), (tuple(t.clone() for t in q13), tuple(t.clone() for t in q2))]
        dsteps4 = max(args.steps, 20) * 5

        def dstep4(i):
            a, b = sets4[i & 1]
            moe_fwd(xd4, idd4, wtd4, a, b, out=outd4, workspace=ws4)

        for i in range(10):
            dstep4(i)
        barrier()
        ev0.record()
        for i in range(dsteps4):
            dstep4(i)
        ev1.record()
        barrier()
        d4_ms = max_over_ranks(ev0.elapsed_time(ev1)) / dsteps4
        ctx.profile_begin(max_marks=dsteps4 * 8 + 8)
        for i in range(dsteps4):
            dstep4(i)
        dst4 = ctx.profile_end()
        ctx.check_device_status()
        wbytes4 = sum(t.numel() * t.element_size() for t in (*q13, *q2)) + 2 * M_DECODE * H * 2
        w4["decode"] = {
            "workload": f"moe_ffn_decode_M256 with {label} weights (pre-quantized, two copies alternated)",
            "ms_per_step": d4_ms, "tokens_per_s": world * M_DECODE / (d4_ms * 1e-3),
            "algorithmic_bytes": wbytes4, "gbs": wbytes4 / (d4_ms * 1e-3) / 1e9,
            "frac_hbm_measured": wbytes4 / (d4_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
            "stage_ms": {k: v[0] / dsteps4 for k, v in dst4.items() if v[1]},
        }
        return w4

    if not args.no_w4a16:
        result["w4a16"] = bench_4bit("W4A16", ctx.quantize_weight_w4, ctx.moe_fwd_w4a16)
        result["fp4a16"] = bench_4bit("FP4A16 (e2m1)", ctx.quantize_weight_fp4, ctx.moe_fwd_fp4a16)

    # ---------------- full-precision backward of the dense projection (QKV shape of the training configuration)
    if not args.no_backward:
        Mb, Nb, Kb = 8192, 5120, 2048
        gen = torch.Generator(device=dev).manual_seed(3000 + rank)
        dyb = torch.randn((Mb, Nb), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        xb = torch.randn((Mb, Kb), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        wb = (torch.randn((Nb, Kb), generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
        bsteps = max(args.steps, 20)
        for _ in range(3):
            ctx.linear_bwd(dyb, xb, wb)
        barrier()
        ev0.record()
        for _ in range(bsteps):
            ctx.linear_bwd(dyb, xb, wb)
        ev1.record()
        barrier()
        b_ms = max_over_ranks(ev0.elapsed_time(ev1)) / bsteps
        ctx.profile_begin(max_marks=bsteps * 4 + 8)
        for _ in range(bsteps):
            ctx.linear_bwd(dyb, xb, wb)
        bst = ctx.profile_end()
        ctx.check_device_status()
        fl = 2.0 * Mb * Nb * Kb
        dx_ms = bst["bwd_dx"][0] / max(bst["bwd_dx"][1], 1)
        dw_ms = bst["bwd_dw"][0] / max(bst["bwd_dw"][1], 1)
        result["backward"] = {
            "workload": (f"straight-through backward of the dense projection, M={Mb} N={Nb} K={Kb} (bf16 masters); "
                         "213 MB of operands and results per step, larger than L2"),
            "ms_per_step": b_ms, "dx_ms": dx_ms, "dw_ms": dw_ms,
            "dx_tflops": fl / (dx_ms * 1e-3) / 1e12, "dw_tflops": fl / (dw_ms * 1e-3) / 1e12,
            "dx_frac_bf16_peak_measured_burst": fl / (dx_ms * 1e-3) / 1e12 / pk["bf16_burst"],
            "dw_frac_bf16_peak_measured_burst": fl / (dw_ms * 1e-3) / 1e12 / pk["bf16_burst"],
        }
        # the expert gate_up projection of the training batch (expert-sorted rows, Zipf group sizes)
        rows = torch.bincount(ids.flatten().to(torch.int64), minlength=E)
        goff = torch.zeros(E + 1, dtype=torch.int32, device=dev)
        goff[1:] = torch.cumsum(rows, 0).to(torch.int32)
        Pg = M_TRAIN * TOPK
        dyg = torch.randn((Pg, 2 * I), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        xg = torch.randn((Pg, H), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        gsteps = max(args.steps // 5, 5)
        for _ in range(2):
            ctx.grouped_linear_bwd(dyg, xg, w13, goff)
        ctx.profile_begin(max_marks=gsteps * 4 + 8)
        for _ in range(gsteps):
            ctx.grouped_linear_bwd(dyg, xg, w13, goff)
        gst = ctx.profile_end()
        ctx.check_device_status()
        gfl = 2.0 * Pg * 2 * I * H
        gdx = gst["bwd_dx"][0] / max(gst["bwd_dx"][1], 1)
        gdw = gst["bwd_dw"][0] / max(gst["bwd_dw"][1], 1)
        result["backward"]["grouped"] = {
            "workload": f"backward of the expert gate_up projection, {Pg} expert-sorted rows, E={E}, N={2 * I}, K={H}",
            "dx_ms": gdx, "dw_ms": gdw, "dx_tflops": gfl / (gdx * 1e-3) / 1e12, "dw_tflops": gfl / (gdw * 1e-3) / 1e12,
            "dx_frac_bf16_peak_measured_sustained": gfl / (gdx * 1e-3) / 1e12 / pk["bf16_sustained"],
            "dw_frac_bf16_peak_measured_sustained": gfl / (gdw * 1e-3) / 1e12 / pk["bf16_sustained"],
        }
        # backward of the whole routed-expert layer on the training batch (activations saved by the forward)
        saved = dict(gate_up=torch.empty((M_TRAIN * TOPK, 2 * I), dtype=torch.bfloat16, device=dev),
                     h=torch.empty((M_TRAIN * TOPK, I), dtype=torch.bfloat16, device=dev))
        ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, out=out, workspace=ws, save=saved)
        gu_saved, h_saved = saved["gate_up"], saved["h"]
        doutb = torch.randn((M_TRAIN, H), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        bws = torch.empty(ctx.lib.qarl_moe_bwd_workspace_bytes(M_TRAIN, H, I, E, TOPK), dtype=torch.uint8, device=dev)
        bout = ctx.moe_bwd(x, ids, wts, w13, w2, gu_saved, h_saved, doutb, workspace=bws)
        msteps = max(args.steps // 5, 5)
        ctx.moe_bwd(x, ids, wts, w13, w2, gu_saved, h_saved, doutb, out=bout, workspace=bws)
        barrier()
        ev0.record()
        for _ in range(msteps):
            ctx.moe_bwd(x, ids, wts, w13, w2, gu_saved, h_saved, doutb, out=bout, workspace=bws)
        ev1.record()
        barrier()
        mb_ms = max_over_ranks(ev0.elapsed_time(ev1)) / msteps
        ctx.profile_begin(max_marks=msteps * 16 + 8)
        for _ in range(msteps):
            ctx.moe_bwd(x, ids, wts, w13, w2, gu_saved, h_saved, doutb, out=bout, workspace=bws)
        mst = ctx.profile_end()
        ctx.check_device_status()
        bfl = 2.0 * M_TRAIN * FLOP_PER_TOKEN
        result["backward"]["moe_layer"] = {
            "workload": f"backward of the routed-expert layer, M={M_TRAIN} (4 grouped bf16 GEMMs + element-wise kernels)",
            "ms_per_step": mb_ms, "tflops": bfl / (mb_ms * 1e-3) / 1e12,
            "frac_bf16_peak_measured_sustained": bfl / (mb_ms * 1e-3) / 1e12 / pk["bf16_sustained"],
            "stage_ms": {k_: v[0] / msteps for k_, v in mst.items() if v[1]},
        }
        # one training step of the layer: quantize + publish-ready codes, low-bit forward that saves its
        # activations, full-precision backward
        def train_step():
            ctx.quantize_weight(w13, w13c, w13s)
            ctx.quantize_weight(w2, w2c, w2s)
            ctx.moe_fwd(x, ids, wts, w13c, w13s, w2c, w2s, out=out, workspace=ws, save=saved)
            ctx.moe_bwd(x, ids, wts, w13, w2, gu_saved, h_saved, doutb, out=bout, workspace=bws)
        train_step()
        barrier()
        ev0.record()
        for _ in range(msteps):
            train_step()
        ev1.record()
        barrier()
        ts_ms = max_over_ranks(ev0.elapsed_time(ev1)) / msteps
        ctx.check_device_status()
        result["backward"]["train_step"] = {
            "workload": f"layer training step, M={M_TRAIN}: weight quantization + FP8 forward (saving gate_up, h) + bf16 backward",
            "ms_per_step": ts_ms, "tokens_per_s": world * M_TRAIN / (ts_ms * 1e-3),
            "tflops": 3.0 * M_TRAIN * FLOP_PER_TOKEN / (ts_ms * 1e-3) / 1e12,
        }
        del gu_saved, h_saved, saved, doutb, bws, bout
        del dyb, xb, wb, dyg, xg

    # ---------------- TBPO sequence-level loss over a packed batch of responses
    if not args.no_tbpo:
        from paper_2604_07853_b200 import inputs as gen_inputs
        lens = gen_inputs.tbpo_lengths(4000 + rank, 4096)
        tcase = [torch.from_numpy(a).to(dev) for a in gen_inputs.tbpo_case(4000 + rank, lens)]
        Tt, Bt = int(tcase[0].shape[0]), int(tcase[4].shape[0])
        tws = torch.empty(max(int(ctx.lib.qarl_tbpo_workspace_bytes(Bt, Tt)), 256), dtype=torch.uint8, device=dev)
        tout = ctx.tbpo_loss(*tcase, workspace=tws)
        tsteps = max(args.steps, 20)
        for _ in range(3):
            ctx.tbpo_loss(*tcase, out=tout, workspace=tws)
        barrier()
        ev0.record()
        for _ in range(tsteps):
            ctx.tbpo_loss(*tcase, out=tout, workspace=tws)
        ev1.record()
        barrier()
        t_ms = max_over_ranks(ev0.elapsed_time(ev1)) / tsteps
        ctx.check_device_status()
        tbytes = 16 * Tt + 8 * (Bt + 1) + 4 * Bt + 28 * Bt
        result["tbpo"] = {
            "workload": f"TBPO loss + per-token gradient, {Bt} packed responses, {Tt} tokens (lognormal lengths, <= 16384); "
                        f"{tbytes / 1e6:.0f} MB per step, larger than L2",
            "ms_per_step": t_ms, "tokens_per_s": world * Tt / (t_ms * 1e-3),
            "algorithmic_bytes": tbytes, "gbs": tbytes / (t_ms * 1e-3) / 1e9,
            "frac_hbm_measured": tbytes / (t_ms * 1e-3) / 1e9 / pk["hbm_gbs"], "launches_per_step": 4,
        }
        del tcase, tout, tws

    # ---------------- decode shape (rollout engine: weights already quantized)
    if not args.no_decode:
        del w13, w2
        _, _, xd, idd, wtd = make_inputs(M_DECODE, 2000 + rank, dev, zipf=False)
        outd = torch.empty((M_DECODE, H), dtype=torch.bfloat16, device=dev)
        # rotate over two copies of the codes so consecutive steps never re-read a resident copy
        sets = [(w13c, w13s, w2c, w2s), (w13c.clone(), w13s.clone(), w2c.clone(), w2s.clone())]
        dsteps = max(args.steps, 20) * 5

        def dstep(i):
            a, b, c, d = sets[i & 1]
            ctx.moe_fwd(xd, idd, wtd, a, b, c, d, out=outd, workspace=ws)

        for i in range(10):
            dstep(i)
        barrier()
        ev0.record()
        for i in range(dsteps):
            dstep(i)
        ev1.record()
        barrier()
        d_ms = max_over_ranks(ev0.elapsed_time(ev1)) / dsteps
        ctx.profile_begin(max_marks=dsteps * 8 + 8)
        for i in range(dsteps):
            dstep(i)
        dst = ctx.profile_end()
        ctx.check_device_status()
        wbytes = w13c.numel() + w2c.numel() + (w13s.numel() + w2s.numel()) * 4 + 2 * M_DECODE * H * 2
        kern_ms = sum(v[0] for v in dst.values()) / dsteps
        result["decode"] = {
            "workload": "moe_ffn_decode_M256 (weights pre-quantized, two weight copies alternated: 1.2 GB > L2)",
            "ms_per_step": d_ms, "tokens_per_s": world * M_DECODE / (d_ms * 1e-3),
            "algorithmic_bytes": wbytes, "gbs": wbytes / (d_ms * 1e-3) / 1e9,
            "frac_hbm_measured": wbytes / (d_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
            "frac_hbm_nominal_8000": wbytes / (d_ms * 1e-3) / 1e9 / 8000.0,
            "stage_ms": {k: v[0] / dsteps for k, v in dst.items() if v[1]},
            "sum_of_kernel_ms": kern_ms,
        }

    # ---------------- CPU oracle baseline (rank 0, N = 1 only), bounded sample
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        n_tokens, n_exp = min(8192, M_TRAIN), 32
        st = cpu_state(4, n_tokens)
        est, raw = cpu_reference_step(st, n_tokens, n_exp)
        # the same sample through the CUDA path (oracle-quantized weights: the quantizers are bit-exact),
        # end to end with no teacher forcing: how far the final bf16 rows are from the oracle's
        def dev_bf16(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(dev)
        got = ctx.moe_fwd(dev_bf16(st["x"]), torch.from_numpy(st["ids"]).to(dev), torch.from_numpy(st["wts"]).to(dev),
                          *[torch.from_numpy(st[k]).to(dev) for k in ("w13c", "w13s", "w2c", "w2s")])
        ctx.check_device_status()
        gb = got.view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int32)
        ob = st["out"].astype(np.int32)
        key = lambda b: np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
        dist = np.abs(key(gb) - key(ob))
        gf = (gb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        of = (ob.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        result["parity_sample"] = {
            "what": f"final bf16 rows of {n_tokens} tokens, CUDA path vs oracle run independently (no teacher forcing)",
            "equal": int((dist == 0).sum()), "one_ulp": int((dist == 1).sum()), "beyond_one_ulp": int((dist > 1).sum()),
            "elements": int(dist.size), "rel_frobenius_error": float(np.linalg.norm(gf - of) / np.linalg.norm(of)),
        }
        result["cpu_baseline"] = {
            "value": M_TRAIN / est, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": (f"oracle quantize_weight on {n_exp} of {E} experts (x{E // n_exp}) + oracle MoE layer on "
                       f"{n_tokens} of {M_TRAIN} tokens (x{M_TRAIN // n_tokens}); {raw:.1f} s of CPU work"),
        }
    elif rank == 0:
        result["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
