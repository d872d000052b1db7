#!/usr/bin/env python
"""Benchmark of the DeaMoE decode layer on B200: us per step and achieved HBM GB/s against the
weight-streaming roofline (unique weight bytes / peak HBM bandwidth).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--batch B] [--shape dsv3|7b]
                    [--schedule auto|plain|staged|fused|dense] [--mode layer|locality|stack|large] [--no-sweep] [--impl reference]

One "step" = one forward of one DeaMoE layer (routing, bucketing, department and private stages,
combine) over one batch of B synthetic tokens.  The headline workload is the DeepSeek-V3-shaped
layer (h 7168, 32 departments x 8 experts, f 2048, private part 1/8 of an expert, top-8, one shared
expert, bf16 weights) at B = 16.  Weights stay resident in HBM; every step streams the unique weights
of its active departments and experts, far more than the L2 holds, and successive steps use
different token batches (different routings).  A 256 MiB buffer is overwritten between steps to
flush L2 (untimed).  Prints ONE JSON line.

With N > 1 every rank runs an independent replica of the same layer on its own GPU -- the path has
no collective -- and the line reports the aggregate.  Under torchrun the ranks are already there
(RANK / LOCAL_RANK / WORLD_SIZE in the environment); invoked plainly with --gpus N > 1 the script
starts the N ranks itself (torchrun on 127.0.0.1) and passes its arguments through.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

PAPER_CONTEXT = {
    "loaded_weights_reduction_max": 0.509,
    "tpot_speedup_7b_a40": 1.33,
    "layer_speedup_dsv3_a40": 2.00,
    "layer_speedup_dsv3_h100": 1.97,
    "note": "the paper's figures (other hardware, its own DeaMoE configuration); context only",
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy read+write)"
    return 6650.0, "fallback (no MEASURED_PEAKS.json: an earlier copy measurement on a B200)"


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1])); power.append(float(p[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def free_port():
    import socket
    sk = socket.socket()
    sk.bind(("127.0.0.1", 0))
    port = sk.getsockname()[1]
    sk.close()
    return port


def spawn_ranks(n, argv):
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one per GPU) the way the driver
    does, on 127.0.0.1, with this script's own arguments; NCCL's communicator log goes to stderr."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd, env=env)


def selftest_cpu(args, rank, world):
    """The multi-rank plumbing without a GPU: process group (gloo), barrier, max over ranks, aggregate."""
    import torch
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("gloo")
        dist.barrier()
    total_ms = max_over_ranks(10.0 * (rank + 1) * args.steps, dist, torch.device("cpu"))
    us = us_per_layer_step(total_ms, args.steps, world)
    if rank == 0:
        print(json.dumps({"selftest": True, "metric": "us_per_step_deamoe_layer", "value": us, "unit": "us",
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3,
                          "scaling": "weak", "slowest_rank_total_ms": total_ms}))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def max_over_ranks(value, dist=None, device=None):
    """The slowest rank's value (all ranks get it); identity without a process group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def us_per_layer_step(total_ms_max, steps, world):
    """Whole-job figure: every rank ran `steps` layer-steps of its own replica in total_ms_max."""
    return total_ms_max * 1e3 / (steps * world)


def pct(xs, q):
    xs = sorted(xs)
    return xs[min(len(xs) - 1, max(0, int(round(q * (len(xs) - 1)))))]


def workload_config(shape, B, schedule):
    """The `config` object of the JSON line; both arms (the CUDA path and --impl reference) print the same."""
    return {"workload": f"{shape.name}-shape DeaMoE layer, decode batch {B} (replica per GPU)",
            "batch": B, "hidden": shape.hidden, "n_dept": shape.n_dept, "experts_per_dept": shape.experts_per_dept,
            "ffn": shape.ffn, "priv": shape.priv, "top_k": shape.top_k, "n_shared": shape.n_shared,
            "schedule": schedule, "l2": "256 MiB buffer overwritten between steps (untimed); "
            "4 rotating token batches", "accumulate": "fp32"}


class HostWeights:
    """Host (numpy) copies of the synthetic layer's matrices for the oracle, generated unit by unit on
    first use (any unit of the counter-based generator can be made alone) and kept."""

    def __init__(self, shape, dev, router=None, shared=None):
        import torch
        from paper_2608_14385_b200 import synth
        self.shape, self.dev, self.synth, self.torch = shape, dev, synth, torch
        self.router = synth.to_numpy(router if router is not None else synth.make_router(shape, 0, dev))
        self.shared = shared
        self.cache = {}

    def unit(self, name, u):
        key = (name, u)
        if key not in self.cache:
            self.cache[key] = self.synth.to_numpy(self.synth.weight_slice(self.shape, name, u, 0, self.dev))
        return self.cache[key]

    def tables(self, depts, experts):
        shape, synth, torch = self.shape, self.synth, self.torch
        w = {"router": self.router}
        for name in ("gate", "up", "down"):
            tab = [None] * shape.n_dept
            for j in depts:
                tab[j] = self.unit(f"dept_{name}", j)
            w[f"dept_{name}"] = tab
            if shape.priv > 0:
                tab = [None] * shape.n_expert
                for i in experts:
                    tab[i] = self.unit(f"priv_{name}", i)
                w[f"priv_{name}"] = tab
            if shape.n_shared:
                key = f"shared_{name}"
                if key not in self.cache:
                    t = self.shared[key] if self.shared else synth.normal(
                        (shape.shared_ffn, shape.hidden), synth.W_STD, 0, f"L0/{key}", self.dev,
                        torch.bfloat16 if shape.weight_dtype else torch.float32)
                    self.cache[key] = synth.to_numpy(t)
                w[key] = self.cache[key]
        return w


def oracle_step_seconds(shape, host, tokens, threads, rows=None):
    """Wall time of the fp64 oracle (as it stands) for ONE whole step on this batch: routing of all B
    tokens once, then Eq. (4) / Eq. (3) for every token row (or only `rows`).  The weights it will touch
    are fetched before the clock starts."""
    from oracle import ref
    from paper_2608_14385_b200 import synth
    cfg = ref.make_config(**shape.asdict())
    tok = synth.to_numpy(tokens)
    ref.set_threads(ref.host_cores())
    sel = ref.route(cfg, host.router, tok)["idx"]
    if rows is not None:
        sel = sel[rows]
    experts = sorted({int(i) for i in sel.reshape(-1)})
    depts = sorted({i // shape.experts_per_dept for i in experts})
    w = host.tables(depts, experts)
    ref.set_threads(threads)
    t0 = time.perf_counter()
    ref.deamoe_forward(cfg, w, tok, rows=rows)
    dt = time.perf_counter() - t0
    ref.set_threads(ref.host_cores())
    return dt


def run_reference(args, shape, rank, world):
    """--impl reference: the oracle on the host cores, rank 0 only.  Every step is one whole layer step
    (all B token rows, routing once), so value x steps is the time the run really spent in the oracle."""
    if rank != 0:
        return
    import torch
    from oracle import ref
    from paper_2608_14385_b200 import synth
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    B = args.batch
    cores = ref.host_cores()
    host = HostWeights(shape, dev)
    times = []
    for step in range(args.warmup + args.steps):
        tokens = synth.make_tokens(shape, B, 100 + step % 4, dev)
        sec = oracle_step_seconds(shape, host, tokens, cores)
        if step >= args.warmup:
            times.append(sec)
    us = statistics.mean(times) * 1e6
    line = {
        "impl": "reference", "metric": "us_per_step_deamoe_layer", "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(shape, B, args.schedule),
        "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle",
                         "sample": f"every step: all {B} token rows of one layer step (routing once), fp64"},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# dram__bytes_read.sum + dram__bytes_write.sum of the weight-streaming launches divided by their algorithmic
# bytes, from the committed one-pass ncu captures of the benchmark's own full-size launches
# (profiles/dram_traffic_full_size_dsv3_b16_b128.md): k_stream at B = 16, and k_dense + k_stream + k_dense at B = 128
DRAM_TRAFFIC_RATIO = 1.0013
DRAM_TRAFFIC_RATIO_DENSE = 1.0127


def read_only_ceiling(binding, torch, dev, gib=4, reps=6):
    """GB/s of a plain vectorised read of a `gib` GiB buffer (the library's deamoe_probe_read kernel),
    best of `reps`, CUDA events: what a read-only HBM stream reaches on this GPU, measured in this run."""
    buf = torch.empty(gib << 30, dtype=torch.uint8, device=dev)
    buf.fill_(1)
    sink = torch.zeros(binding.PROBE_BLOCKS, dtype=torch.int32, device=dev)
    best = 0.0
    for i in range(reps + 2):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        binding.probe_read(buf, sink)
        b.record()
        torch.cuda.synchronize()
        if i >= 2:
            best = max(best, buf.numel() / (a.elapsed_time(b) * 1e-3) / 1e9)
    del buf
    torch.cuda.empty_cache()
    return best


def stream_kernel_ms(layer, batches, steps, flush, torch):
    """Per-step duration (ms) of the weight-streaming launches, from the library's own event pair."""
    layer.profile(True)
    out = torch.empty_like(batches[0])
    ms = []
    for i in range(steps + 2):
        flush.add_(1)
        layer.forward(batches[i % len(batches)], out)
        t = layer.last_stream_ms()
        if i >= 2:
            ms.append(t)
    layer.profile(False)
    return ms


def time_layer(layer, batches, steps, warmup, flush, torch, barrier):
    """Per-step CUDA-event times (ms) of layer.forward over rotating token batches."""
    outs = [torch.empty_like(b) for b in batches]
    for i in range(warmup):
        flush.add_(1)
        layer.forward(batches[i % len(batches)], outs[i % len(batches)])
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    launches = 0
    torch.cuda.synchronize()
    barrier()
    for i in range(steps):
        flush.add_(1)                      # overwrite 256 MiB: evicts the previous step from L2
        ev[i][0].record()
        layer.forward(batches[i % len(batches)], outs[i % len(batches)])
        ev[i][1].record()
        launches += layer.last_launches
    torch.cuda.synchronize()
    barrier()
    return [a.elapsed_time(b) for a, b in ev], launches


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--shape", default="dsv3")
    ap.add_argument("--schedule", default="auto", choices=["auto", "plain", "staged", "fused", "dense"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true", help="skip the batch sweep and the vanilla comparator")
    ap.add_argument("--no-cpu", action="store_true", help="skip the timed CPU oracle")
    ap.add_argument("--mode", default="layer", choices=["layer", "locality", "stack", "large"],
                    help="layer: the contract line (default); locality: routing-locality sweep on the DeepSeek-V3 "
                         "shape; stack: 32 consecutive 7B-class layers with a residual add, DeaMoE vs vanilla; "
                         "large: 32-128 tokens on the DeepSeek-V3 shape, streaming vs dense (tcgen05) schedule")
    ap.add_argument("--shard", default="replica", choices=["replica", "dept"],
                    help="replica (default): every rank runs its own copy of the layer, no collective; dept: ONE layer "
                         "spread over the ranks by department (each rank holds its departments' weights, computes "
                         "their partial sum, one NCCL all-reduce of [B, h] fp32 completes Eq. (3)): strong scaling")
    ap.add_argument("--selftest-cpu", action="store_true",
                    help="no GPU work: every rank reports a fixed made-up duration through the same rank start-up, "
                         "barrier and max-over-ranks code (gloo); used by the CPU tests of the multi-rank path")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))

    from paper_2608_14385_b200 import synth
    shape = synth.SHAPES[args.shape]
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, shape, rank, world)
        return
    if args.selftest_cpu:
        selftest_cpu(args, rank, world)
        return

    import torch
    from paper_2608_14385_b200 import binding
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()

    sched = {"auto": binding.SCHED_AUTO, "plain": binding.SCHED_PLAIN, "staged": binding.SCHED_STAGED,
             "fused": binding.SCHED_FUSED, "dense": binding.SCHED_DENSE}[args.schedule]
    peak, peak_src = measured_peaks()
    if args.mode != "layer":
        if rank == 0:
            fn = {"locality": locality_sweep, "stack": stack_bench, "large": large_batch_sweep}[args.mode]
            print(json.dumps(fn(args, sched, peak, torch, dev)))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    if args.shard == "dept":
        line = sharded_bench(args, shape, sched, peak, peak_src, torch, dev, dist, rank, local, world)
        if rank == 0:
            print(json.dumps(line))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    B = args.batch
    # (sized for the largest batch of the sweep; from 32 tokens on AUTO takes the dense schedule)
    max_batch = max(64 if shape.name in synth.PAPER_BASELINES else (128 if shape.name == "dsv3" and not args.no_sweep else 32), B)
    w = synth.make_deamoe_weights(shape, 0, dev)
    layer = binding.Layer(shape, w, max_batch, sched)
    router = w["router"]
    shared = {k: v for k, v in w.items() if k.startswith("shared_")}
    del w
    torch.cuda.empty_cache()
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    NB = 4
    batches = [synth.make_tokens(shape, B, 100 + i, dev) for i in range(NB)]
    ubytes = []
    for b in batches:
        layer.forward(b)
        ubytes.append(layer.stats()["unique_weight_bytes"])

    read_gbs = read_only_ceiling(binding, torch, dev)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.5)      # nvidia-smi needs a moment before its first sample
    times_ms, launches = time_layer(layer, batches, args.steps, args.warmup, flush, torch, barrier)
    # keep the GPU under the same load a little longer so the sampler sees it (untimed)
    t_end = time.time() + 0.6
    while time.time() < t_end:
        layer.forward(batches[0])
    torch.cuda.synchronize()
    clocks = sampler.stop()
    # the same steps with nothing overwritten in between, where a step's own weights are several times the L2 (the
    # timing rules' other choice: inputs larger than L2): what a decode loop over this one layer sees, with the
    # kernels' code and the 7 MB router still resident.  Context beside `value`, which keeps the overwrite.
    steady_us = None
    if min(ubytes) > 4 * (126 << 20):
        class _Keep:
            def add_(self, x):
                pass
        t2, _ = time_layer(layer, batches, max(8, args.steps // 2), 3, _Keep(), torch, lambda: None)
        steady_us = pct(t2, 0.5) * 1e3
    total_ms = max_over_ranks(sum(times_ms), dist, dev)
    # aggregate: layer-steps processed by all ranks per unit time -> us per layer-step
    us_per_step = us_per_layer_step(total_ms, args.steps, world)
    step_bytes = [ubytes[i % NB] for i in range(args.steps)]
    gbs = [bts / (ms * 1e-3) / 1e9 for bts, ms in zip(step_bytes, times_ms)]
    mean_bytes = statistics.mean(step_bytes)

    # dominant kernel (weight streaming): events recorded by the library, on the stream it launches
    # on, around its k_stream launch(es); algorithmic bytes = the step's unique weight bytes minus
    # the fp32 router matrix (read by the routing kernel, outside the pair of events)
    kern = stream_kernel_ms(layer, batches, args.steps, flush, torch) if args.schedule != "plain" else None
    router_bytes = shape.n_expert * shape.hidden * 4
    if kern:
        k_ms = statistics.mean(kern)
        alg = statistics.mean(step_bytes) - router_bytes
        achieved = alg / (k_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": alg * DRAM_TRAFFIC_RATIO,
                "traffic_note": "ESTIMATE for this run: its algorithmic bytes x 1.0013, the (dram read + write) / algorithmic "
                                "ratio that ncu measured on this workload's own k_stream launches (one-pass capture of four "
                                "full-size launches at B = 16, profiles/dram_traffic_full_size_dsv3_b16_b128.md)",
                "kernel": "k_stream (the weight-streaming launch(es) of one step)",
                "kernel_ms": k_ms, "peak_source": peak_src, "algorithmic_bytes_per_launch": alg,
                "read_only_ceiling_gbs": read_gbs,
                "read_only_ceiling_note": "plain 16-byte-load read of 4 GiB by deamoe_probe_read, best of 6, this run; "
                                          "`peak` is a read+write copy figure, which a read-only stream may exceed",
                "frac_of_read_only_ceiling": achieved / read_gbs if read_gbs else None,
                "frac_of_nominal_8TBs": achieved / 8000.0}
        if args.schedule == "dense" or (args.schedule == "auto" and B >= binding.dense_min_batch(shape)):
            # dense schedule: the pair of events brackets the gather kernel and k_dense, k_stream, k_dense (a chain that hands over through counters)
            roof["kernel"] = "k_dense + k_stream + k_dense (the three weight-streaming launches of a dense step)"
            roof["traffic_note"] = ("ESTIMATE for this run: its algorithmic bytes x 1.0127, the ratio ncu measured on the three "
                                    "full-size launches of a dense step at B = 128 "
                                    "(profiles/dram_traffic_full_size_dsv3_b16_b128.md)")
            roof["traffic"] = alg * DRAM_TRAFFIC_RATIO_DENSE
    else:
        achieved = mean_bytes / (statistics.mean(times_ms) * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None, "kernel": "whole step (plain schedule has no single dominant kernel)",
                "peak_source": peak_src, "algorithmic_bytes_per_step": mean_bytes}

    # end to end through the public host-buffer entry point
    host_in = [b.cpu().pin_memory() for b in batches]
    host_out = torch.empty_like(host_in[0]).pin_memory()
    for i in range(3):
        layer.forward_host(host_in[i % NB], host_out)
    e2e_t = []
    for i in range(args.steps):
        flush.add_(1)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        layer.forward_host(host_in[i % NB], host_out)
        e2e_t.append(time.perf_counter() - t0)
    io_bytes = B * shape.hidden * (2 if shape.act_dtype else 4)
    e2e_us = max_over_ranks(statistics.mean(e2e_t) * 1e6, dist, dev) / world

    line = {
        "metric": "us_per_step_deamoe_layer", "value": us_per_step, "unit": "us", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us_per_step / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if shape.weight_dtype else "f32",
        "data": "synthetic",
        "config": workload_config(shape, B, args.schedule),
        "us_per_step_p10_p50_p90": [pct(times_ms, 0.1) * 1e3, pct(times_ms, 0.5) * 1e3, pct(times_ms, 0.9) * 1e3],
        "hbm_gbs_on_unique_bytes": {"mean": statistics.mean(gbs), "p50": pct(gbs, 0.5),
                                    "frac_of_measured_peak": statistics.mean(gbs) / peak,
                                    "frac_of_nominal_8TBs": statistics.mean(gbs) / 8000.0},
        "unique_weight_mb_per_step": mean_bytes / 1e6,
        "us_per_step_without_l2_overwrite_p50": steady_us,
        "clocks": clocks,
        "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": io_bytes, "d2h_bytes_per_step": io_bytes},
        "gpu_launches": launches,
        "roofline": roof,
        "paper_context": PAPER_CONTEXT,
    }

    if rank == 0 and not args.no_sweep:
        if shape.name in synth.PAPER_BASELINES:
            line["sweep"] = paper_row_sweep(args, shape, layer, flush, sched, peak, torch, dev)
        else:
            line["sweep"] = sweep(args, shape, layer, router, shared, flush, sched, peak, torch, dev)
    if rank == 0 and not args.no_cpu:
        from oracle import ref
        host = HostWeights(shape, dev, router=router, shared=shared)
        cores = ref.host_cores()
        sec = oracle_step_seconds(shape, host, batches[0], cores)
        few = list(range(min(B, 2)))
        one = oracle_step_seconds(shape, host, batches[0], 1, rows=few)
        line["cpu_baseline"] = {"value": sec * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
                                "sample": f"one whole layer step: all {B} token rows, routing once, fp64",
                                "one_core_us_per_token_row": one * 1e6 / len(few),
                                "one_core_sample": f"{len(few)} of {B} token rows on one core (not scaled)"}
    if rank == 0 and not args.no_sweep and shape.name == "dsv3":
        locality = locality_rows(shape, layer, router, flush, peak, torch, dev, cs=(1, 2, 4, 8), batches_list=(1, 16), steps=10)
        layer.close()
        layer = None
        torch.cuda.empty_cache()
        line["other_workloads"] = other_workloads(args, sched, peak, torch, dev, flush)
        line["other_workloads"]["locality_dsv3"] = {
            "workload": "dsv3-shape DeaMoE layer, every token's top-8 planted in exactly c departments (configuration 4)",
            "rows": locality}
    if layer is not None:
        layer.close()
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def sharded_bench(args, shape, sched, peak, peak_src, torch, dev, dist, rank, local, world):
    """--shard dept: one layer spread over the ranks by department (paper Section 3.1: a department and
    its experts' private matrices are an independent unit).  A step = forward_partial on every rank, one
    all-reduce (NCCL) of the [B, h] fp32 partial sums, finish_partial.  Total work is fixed as N grows."""
    from paper_2608_14385_b200 import binding, shard, synth
    B = args.batch
    my_shape, (lo, hi) = shard.slice_shape(shape, rank, world)
    w = synth.make_deamoe_weights(my_shape, 0, dev, dept_range=(lo, hi))
    layer = binding.Layer(my_shape, w, max(B, 32), sched, dept_range=(lo, hi))
    del w
    torch.cuda.empty_cache()
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    NB = 4
    batches = [synth.make_tokens(shape, B, 100 + i, dev) for i in range(NB)]
    partial = torch.empty((B, shape.hidden), dtype=torch.float32, device=dev)
    outs = [torch.empty_like(b) for b in batches]

    def step(i):
        layer.forward_partial(batches[i % NB], partial)
        if dist is not None:
            dist.all_reduce(partial)
        layer.finish_partial(partial, batches[i % NB], outs[i % NB])

    ubytes = []
    for i in range(NB):
        step(i)
        t = torch.tensor([float(layer.stats()["unique_weight_bytes"])], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(t)
        ubytes.append(float(t.item()))
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.5)
    for i in range(args.warmup):
        flush.add_(1)
        step(i)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    for i in range(args.steps):
        flush.add_(1)
        ev[i][0].record()
        step(i)
        ev[i][1].record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    times_ms = [a.elapsed_time(b) for a, b in ev]
    clocks = sampler.stop()
    total_ms = max_over_ranks(sum(times_ms), dist, dev)
    us = total_ms * 1e3 / args.steps
    mean_bytes = statistics.mean(ubytes[i % NB] for i in range(args.steps))
    launches = args.steps * (layer.last_launches + 1)
    layer.close()
    cfg = workload_config(shape, B, args.schedule)
    cfg["workload"] = f"{shape.name}-shape DeaMoE layer, decode batch {B}, ONE layer sharded by department over {world} GPU(s)"
    cfg["parallelism"] = f"dept-shard x{world}: departments [{lo}, {hi}) on rank {rank}; all-reduce of [B, h] fp32"
    return {"metric": "us_per_step_deamoe_layer", "value": us, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16" if shape.weight_dtype else "f32", "data": "synthetic", "config": cfg,
            "unique_weight_mb_per_step_all_ranks": mean_bytes / 1e6,
            "hbm_gbs_on_unique_bytes_all_ranks": mean_bytes / (us * 1e-6) / 1e9,
            "frac_of_measured_peak_per_gpu": mean_bytes / (us * 1e-6) / 1e9 / (peak * world),
            "clocks": clocks, "gpu_launches": launches, "peak_source": peak_src}


def paper_row_sweep(args, shape, layer, flush, sched, peak, torch, dev, batches_list=(4, 8, 16, 32, 64), steps=None):
    """The paper's own DeepSeek-V3-matched DeaMoE row (8 x 108 experts, square private matrices, top-10 in
    at most 5 departments) against the model it was matched to: a standard 256-expert top-8 MoE layer of
    the DeepSeek-V3 shape (no shared expert, as in the paper's Table 1 accounting), same token counts.
    Reports time, unique bytes, their ratio (the quantity of the paper's Fig. 2) and the speed-up."""
    import dataclasses
    from paper_2608_14385_b200 import binding, synth
    steps = steps or max(10, args.steps // 2)
    res = {}
    for B in batches_list:
        bs = [synth.make_tokens(shape, B, 100 + i, dev) for i in range(4)]
        ub = []
        for b in bs:
            layer.forward(b)
            ub.append(layer.stats()["unique_weight_bytes"])
        t, _ = time_layer(layer, bs, steps, 3, flush, torch, lambda: None)
        res[B] = {"batch": B, "deamoe_us": pct(t, 0.5) * 1e3, "deamoe_mb": statistics.mean(ub) / 1e6}
    base = synth.PAPER_BASELINES[shape.name]
    vw = synth.make_vanilla_weights(base, 0, dev)
    vl = binding.Layer(base, vw, 64, sched, vanilla=True)
    del vw
    torch.cuda.empty_cache()
    out = []
    for B in batches_list:
        bs = [synth.make_tokens(base, B, 100 + i, dev) for i in range(4)]
        ub = []
        for b in bs:
            vl.forward(b)
            ub.append(vl.stats()["unique_weight_bytes"])
        t, _ = time_layer(vl, bs, steps, 3, flush, torch, lambda: None)
        r = res[B]
        r["baseline_moe_us"] = pct(t, 0.5) * 1e3
        r["baseline_moe_mb"] = statistics.mean(ub) / 1e6
        r["deamoe_gbs"] = r["deamoe_mb"] / r["deamoe_us"] * 1e3
        r["baseline_moe_gbs"] = r["baseline_moe_mb"] / r["baseline_moe_us"] * 1e3
        r["deamoe_frac_of_measured_peak"] = r["deamoe_gbs"] / peak
        r["loaded_bytes_ratio_deamoe_over_baseline"] = r["deamoe_mb"] / r["baseline_moe_mb"]
        r["speedup_vs_baseline_moe"] = r["baseline_moe_us"] / r["deamoe_us"]
        out.append(r)
    vl.close()
    ctx = ("expected loaded-weights ratio 0.491 .. 0.628 over 4 .. 64 tokens (Section 3.3, Fig. 2); peak layer "
           "speed-up 2.00x (A40) / 1.97x (H100)") if shape.name == "dsv3-paper" else \
          "Fig. 2 shows this model's loaded-weights ratio as a curve only (no printed numbers)"
    return {"rows": out, "baseline": {"name": base.name, "n_expert": base.n_expert, "top_k": base.top_k},
            "paper_context": ctx}


def locality_rows(shape, layer, router, flush, peak, torch, dev, cs, batches_list, steps):
    """Rows of the routing-locality sweep on an existing layer: every token's top-k is planted (through the
    real router) in exactly c departments (c = 0: no planting, uniform routing).  Unique bytes are set against
    the closed form |D| ~ m (1 - (1 - c/m)^B) with k B distinct experts at most."""
    from paper_2608_14385_b200 import synth
    m, k = shape.n_dept, shape.top_k
    dept_b = 3 * shape.hidden * shape.ffn * 2
    exp_b = 3 * shape.priv * shape.ffn * 2
    fixed_b = shape.n_shared * 3 * shape.hidden * shape.shared_ffn * 2 + shape.n_expert * shape.hidden * 4
    rows = []
    for c in cs:
        for B in batches_list:
            bs = []
            for i in range(4):
                t = synth.make_tokens(shape, B, 200 + i, dev)
                if c:
                    t, _ = synth.plant_locality(shape, router, t, c, seed=10 * c + i)
                bs.append(t)
            ub, nd, ne = [], [], []
            for b in bs:
                layer.forward(b)
                st = layer.stats()
                ub.append(st["unique_weight_bytes"]); nd.append(st["active_dept"]); ne.append(st["active_expert"])
            t_ms, _ = time_layer(layer, bs, steps, 3, flush, torch, lambda: None)
            us = pct(t_ms, 0.5) * 1e3
            mb = statistics.mean(ub) / 1e6
            row = {"c": c if c else "uniform", "batch": B, "us": us, "unique_mb": mb, "gbs": mb / us * 1e3,
                   "frac_of_measured_peak": mb / us * 1e3 / peak, "active_dept": statistics.mean(nd),
                   "active_expert": statistics.mean(ne)}
            if c:
                e_d = m * (1.0 - (1.0 - c / m) ** B)
                e_e = shape.n_expert * (1.0 - (1.0 - k / shape.n_expert) ** B)   # experts uniform over all n
                row["closed_form_mb"] = (e_d * dept_b + e_e * exp_b + fixed_b) / 1e6
                row["closed_form_active_dept"] = e_d
            rows.append(row)
    return rows


def locality_sweep(args, sched, peak, torch, dev):
    """Routing-locality sweep on the DeepSeek-V3 shape (BASELINE configuration 4): c = 1, 2, 4, 8 and uniform
    routing at B = 1, 4, 16, 32."""
    from paper_2608_14385_b200 import binding, synth
    shape = synth.DSV3
    w = synth.make_deamoe_weights(shape, 0, dev)
    layer = binding.Layer(shape, w, 32, sched)
    router = w["router"]
    del w
    torch.cuda.empty_cache()
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    rows = locality_rows(shape, layer, router, flush, peak, torch, dev, cs=(1, 2, 4, 8, 0), batches_list=(1, 4, 16, 32),
                         steps=max(10, args.steps // 2))
    layer.close()
    return {"metric": "routing_locality_sweep", "unit": "us", "shape": shape.name, "data": "synthetic",
            "config": {"workload": "dsv3-shape DeaMoE layer, top-8 planted in c departments per token",
                       "l2": "256 MiB buffer overwritten between steps (untimed)"},
            "rows": rows}


def stack_bench(args, sched, peak, torch, dev, steps=None):
    """32 consecutive 7B-class layers, x <- x + Layer_l(x), every layer with its own seeded weights;
    MoE time per decode step of the DeaMoE stack and of the vanilla-MoE stack at B = 1 and 8.  The stacks
    (6.6 GB and 17.7 GB) are far larger than L2, so no flush is needed between steps.  A step (the
    128 kernels of the 32 layers) is captured once in a CUDA graph and timed as ONE graph launch per
    step, the way a serving runtime replays a decode step (Section 5 of the paper); the same step
    enqueued kernel by kernel is reported beside it."""
    import dataclasses
    from paper_2608_14385_b200 import binding, synth
    shape = dataclasses.replace(synth.MOE7B, residual=1)
    n_layers = 32
    steps = steps or max(10, args.steps // 2)
    out = {"metric": "us_per_decode_step_moe_stack", "unit": "us", "layers": n_layers, "shape": shape.name,
           "data": "synthetic", "config": {"workload": "stack of 32 7B-class layers with residual add",
                                           "launch": "one CUDA-graph replay per step",
                                           "l2": "stack larger than L2, no flush"}, "rows": []}
    res = {}
    for vanilla in (False, True):
        layers = []
        for l in range(n_layers):
            w = (synth.make_vanilla_weights if vanilla else synth.make_deamoe_weights)(shape, 0, dev, layer=l)
            layers.append(binding.Layer(shape, w, 8, sched, vanilla=vanilla))
            del w
        torch.cuda.empty_cache()
        for B in (1, 8):
            # tokens scaled by 1/16: with N(0,1) tokens the vanilla stack (gain ~0.6 per layer, quadratic in |x|)
            # overflows bf16 within 32 layers without a normalisation; routing (an arg-max) is scale-invariant
            xs = [(synth.make_tokens(shape, B, 300 + i, dev).float() / 16).to(torch.bfloat16) for i in range(4)]
            x_in = xs[0].clone()
            bufs = [torch.empty_like(xs[0]), torch.empty_like(xs[0])]

            def step():
                cur = x_in
                for l, layer in enumerate(layers):      # enqueued back to back, no host synchronisation
                    layer.forward(cur, bufs[l & 1])
                    cur = bufs[l & 1]
                return cur
            for i in range(3):
                x_in.copy_(xs[i % 4])
                step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            torch.cuda.synchronize()

            def timed(run):
                ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
                for i in range(2):
                    x_in.copy_(xs[i % 4])
                    run()
                torch.cuda.synchronize()
                for i in range(steps):
                    x_in.copy_(xs[i % 4])
                    ev[i][0].record()
                    run()
                    ev[i][1].record()
                torch.cuda.synchronize()
                return pct([a.elapsed_time(b) for a, b in ev], 0.5) * 1e3
            t_graph = timed(graph.replay)
            t_enq = timed(step)
            ub = 0
            for layer in layers:
                ub += layer.stats()["unique_weight_bytes"]
            ok = all(layer.stats()["device_status"] == 0 for layer in layers)
            finite = bool(torch.isfinite(bufs[(n_layers - 1) & 1].float()).all())
            res[(vanilla, B)] = (t_graph, ub / 1e6, finite and ok, t_enq)
            del graph
        for layer in layers:
            layer.close()
        del layers
        torch.cuda.empty_cache()
    for B in (1, 8):
        d_us, d_mb, d_fin, d_enq = res[(False, B)]
        v_us, v_mb, v_fin, v_enq = res[(True, B)]
        out["rows"].append({"batch": B, "deamoe_us": d_us, "deamoe_mb_last_step": d_mb, "deamoe_gbs": d_mb / d_us * 1e3,
                            "vanilla_us": v_us, "vanilla_mb_last_step": v_mb, "vanilla_gbs": v_mb / v_us * 1e3,
                            "speedup_vs_vanilla": v_us / d_us, "byte_ratio_vanilla_over_deamoe": v_mb / d_mb,
                            "deamoe_us_per_layer": d_us / n_layers, "outputs_finite_and_status_ok": d_fin and v_fin,
                            "deamoe_us_enqueued_kernel_by_kernel": d_enq, "vanilla_us_enqueued_kernel_by_kernel": v_enq})
    return out


def other_workloads(args, sched, peak, torch, dev, flush):
    """Compact rows for the other benchmark configurations, run after the headline so that one default
    invocation measures them all: one 7B-class layer (configuration 2), the stack of 32 such layers
    (configuration 5), the paper's own DeepSeek-V3-matched row of Table 1 with group-limited routing, and the
    table's other four rows."""
    from paper_2608_14385_b200 import binding, synth
    t0 = time.time()
    out = {}
    shape = synth.MOE7B
    w = synth.make_deamoe_weights(shape, 0, dev)
    layer = binding.Layer(shape, w, 16, sched)
    router = w["router"]
    del w
    rows = sweep(args, shape, layer, router, {}, flush, sched, peak, torch, dev, steps=12)
    layer.close()
    torch.cuda.empty_cache()
    out["7b_layer"] = {"workload": "7b-shape DeaMoE layer vs vanilla MoE, L2 overwritten between steps", "rows": rows}
    out["stack_32x7b"] = stack_bench(args, sched, peak, torch, dev, steps=10)
    shape = synth.DSV3_PAPER
    w = synth.make_deamoe_weights(shape, 0, dev)
    layer = binding.Layer(shape, w, 64, sched)
    del w
    torch.cuda.empty_cache()
    out["dsv3_paper_row"] = paper_row_sweep(args, shape, layer, flush, sched, peak, torch, dev, batches_list=(4, 16, 64),
                                            steps=10)
    layer.close()
    torch.cuda.empty_cache()
    # the other rows of the paper's Table 1, each against the standard MoE layer it was matched to
    out["table1_rows"] = {}
    for name in ("dsv2-paper", "qwen3-paper", "kimi-k2-paper", "b7-paper"):
        shape = synth.SHAPES[name]
        w = synth.make_deamoe_weights(shape, 0, dev)
        layer = binding.Layer(shape, w, 64, sched)
        del w
        torch.cuda.empty_cache()
        out["table1_rows"][name] = paper_row_sweep(args, shape, layer, flush, sched, peak, torch, dev,
                                                   batches_list=(4, 16, 64), steps=8)
        layer.close()
        torch.cuda.empty_cache()
    out["seconds"] = time.time() - t0
    return out


def large_batch_sweep(args, sched, peak, torch, dev):
    """48 to 128 tokens on the DeepSeek-V3 shape (the upper half of the paper's 4-128 token range),
    where a department's bucket is a dense tile: the streaming schedule (mma.sync), the dense
    schedule (tcgen05 kernels for the department and shared-expert matrices), what AUTO picks, and the
    in-library vanilla MoE."""
    from paper_2608_14385_b200 import binding, synth
    shape = synth.SHAPES["dsv3"]
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    steps = max(10, args.steps // 2)
    w = synth.make_deamoe_weights(shape, 0, dev)
    router = w["router"]
    layers = {"streaming": binding.Layer(shape, w, 128, binding.SCHED_FUSED),
              "dense": binding.Layer(shape, w, 128, binding.SCHED_DENSE),
              "auto": binding.Layer(shape, w, 128, binding.SCHED_AUTO)}
    del w
    torch.cuda.empty_cache()
    rows = []
    batches_list = [32, 48, 64, 96, 128]
    for B in batches_list:
        bs = [synth.make_tokens(shape, B, 100 + i, dev) for i in range(4)]
        r = {"batch": B}
        for name, layer in layers.items():
            ub = []
            for b in bs:
                layer.forward(b)
                ub.append(layer.stats()["unique_weight_bytes"])
            t, _ = time_layer(layer, bs, steps, 3, flush, torch, lambda: None)
            r[name + "_us"] = pct(t, 0.5) * 1e3
            r["deamoe_mb"] = statistics.mean(ub) / 1e6
        r["auto_gbs"] = r["deamoe_mb"] / r["auto_us"] * 1e3
        r["auto_frac_of_measured_peak"] = r["auto_gbs"] / peak
        rows.append(r)
    for layer in layers.values():
        layer.close()
    torch.cuda.empty_cache()
    vw = synth.make_vanilla_weights(shape, 0, dev, router=router)
    vl = binding.Layer(shape, vw, 128, binding.SCHED_AUTO, vanilla=True)
    del vw
    torch.cuda.empty_cache()
    for r in rows:
        bs = [synth.make_tokens(shape, r["batch"], 100 + i, dev) for i in range(4)]
        ub = []
        for b in bs:
            vl.forward(b)
            ub.append(vl.stats()["unique_weight_bytes"])
        t, _ = time_layer(vl, bs, steps, 3, flush, torch, lambda: None)
        r["vanilla_us"] = pct(t, 0.5) * 1e3
        r["vanilla_mb"] = statistics.mean(ub) / 1e6
        r["speedup_vs_vanilla"] = r["vanilla_us"] / r["auto_us"]
        r["byte_ratio_vanilla_over_deamoe"] = r["vanilla_mb"] / r["deamoe_mb"]
    vl.close()
    return {"metric": "large_batch_sweep", "unit": "us", "shape": shape.name, "data": "synthetic", "dtype": "bf16",
            "l2": "256 MiB buffer overwritten between steps", "peak_gbs_measured": peak, "rows": rows}


def sweep(args, shape, layer, router, shared, flush, sched, peak, torch, dev, steps=None):
    """DeaMoE layer and the in-library vanilla MoE at the same shape over the batch range."""
    from paper_2608_14385_b200 import binding, synth
    out = []
    batches_list = [1, 2, 4, 8, 16, 32, 64, 128] if shape.name == "dsv3" else [1, 4, 16]
    steps = steps or max(10, args.steps // 2)
    res = {}
    for B in batches_list:
        bs = [synth.make_tokens(shape, B, 100 + i, dev) for i in range(4)]
        ub = []
        for b in bs:
            layer.forward(b)
            ub.append(layer.stats()["unique_weight_bytes"])
        t, _ = time_layer(layer, bs, steps, 3, flush, torch, lambda: None)
        res[B] = {"batch": B, "deamoe_us": pct(t, 0.5) * 1e3, "deamoe_mb": statistics.mean(ub) / 1e6}
    vw = synth.make_vanilla_weights(shape, 0, dev, router=router)
    vl = binding.Layer(shape, vw, max(batches_list), sched, vanilla=True)
    del vw
    torch.cuda.empty_cache()
    for B in batches_list:
        bs = [synth.make_tokens(shape, B, 100 + i, dev) for i in range(4)]
        ub = []
        for b in bs:
            vl.forward(b)
            ub.append(vl.stats()["unique_weight_bytes"])
        t, _ = time_layer(vl, bs, steps, 3, flush, torch, lambda: None)
        r = res[B]
        r["vanilla_us"] = pct(t, 0.5) * 1e3
        r["vanilla_mb"] = statistics.mean(ub) / 1e6
        r["deamoe_gbs"] = r["deamoe_mb"] / r["deamoe_us"] * 1e3
        r["vanilla_gbs"] = r["vanilla_mb"] / r["vanilla_us"] * 1e3
        r["deamoe_frac_of_measured_peak"] = r["deamoe_gbs"] / peak
        r["speedup_vs_vanilla"] = r["vanilla_us"] / r["deamoe_us"]
        r["byte_ratio_vanilla_over_deamoe"] = r["vanilla_mb"] / r["deamoe_mb"]
        out.append(r)
    vl.close()
    return out


if __name__ == "__main__":
    main()
