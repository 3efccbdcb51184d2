"""Benchmark of batched draft-tree verification (SpecInfer + Traversal Verification) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole verification path over one batch of synthetic draft trees: every
algorithm the workload lists (SpecInfer, Traversal Verification) is run once on the batch through
the C-ABI library, logits already resident in HBM.  Consecutive calls use different input copies so
that more than the L2 capacity is touched before a copy is read again (reads come from HBM).
The timed block of K steps is repeated R times; the median block gives ``ms_per_step`` and ``value``,
the fastest and slowest are reported beside it.  The row statistics kernel -- the one pass over the
logits in HBM, the kernel the roofline is about -- is also timed by itself.
One JSON line is printed by rank 0.

``--impl reference`` times the CPU checker (``oracle/``) on the host cores instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified tree-nodes/sec"
UNIT = "nodes/s"
L2_BYTES = 132_644_864
ROTATE_BYTES = 4 * L2_BYTES          # bytes touched before an input copy is read again
# The dominant kernel is the row statistics kernel: it is the only one that reads the logits from HBM
# (every logit once), and both verifiers start with it.
STAT_KERNEL = {False: "stream::spec_row_partial_kernel (row statistics: the one pass over the logits in HBM)",
               True: "trunc::spec_row_trunc_kernel (+ rowstat::spec_row_stat_kernel for the rows it leaves over)"}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of that kernel from the ncu captures summarised
# under profiles/ (cold L2).  Workloads without a capture: null.
TRAFFIC_BYTES = {"cfg2_llama3_b8": 69_799_168 + 626_432}
# the same counters summed over the kernels of a whole call, captured in one pass without cache flushes between
# the kernels (profiles/per_config.md): the second kernel of a call finds most of its rows in L2
TRAFFIC_CALL_BYTES = {"cfg2_llama3_b8": {"specinfer": 70_810_000 + 90_000, "traversal": 70_810_000 + 9_200_000}}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="cfg2_llama3_b8")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU work spent on the cpu_baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="enqueue every call from the host instead of replaying CUDA graphs")
    ap.add_argument("--repeats", type=int, default=15, help="timed blocks of --steps steps (median reported)")
    ap.add_argument("--gen", default="cpu", choices=["cpu", "cuda"],
                    help="where the synthetic batches are drawn: cpu gives the same batch for a seed on every machine "
                         "and on both arms; cuda is faster for the largest workloads")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------
# clocks: sample nvidia-smi while the timed region runs
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower() == "active":
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CPU checker legs
# ---------------------------------------------------------------------------------------------
def oracle_step(oracle, host_arrays, w):
    """One pass of the CPU checker over one batch: every algorithm of the workload."""
    inp = oracle.TreeInputs(host_arrays["target_logits"], host_arrays["draft_logits"], host_arrays["parent"],
                            host_arrays["token"], host_arrays["u_accept"], host_arrays["u_bonus"],
                            temperature=w.temperature, top_k=w.top_k, top_p=w.top_p)
    for algo in w.algorithms:
        (oracle.verify_specinfer if algo == "specinfer" else oracle.verify_traversal)(inp)


def _time_oracle(oracle, host, w, seconds: float):
    """Passes of the checker over one batch for about ``seconds``: (passes, wall seconds)."""
    n, t0 = 0, time.perf_counter()
    while True:
        oracle_step(oracle, host, w)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or n >= 10000:
            return n, dt


def cpu_baseline(w, seconds: float) -> dict:
    """The CPU checker as it stands on the host cores: all threads, then one thread, on the same batch."""
    import oracle
    from paper_2602_16994_b200 import synth
    oracle.build()
    host = synth.make_batch(w, seed=0, device="cpu").numpy()
    cores = oracle.max_threads()
    oracle_step(oracle, host, w)                       # warm-up (page-in, thread pool)
    n, dt = _time_oracle(oracle, host, w, seconds)
    nodes = w.draft_nodes() * len(w.algorithms)
    oracle.set_threads(1)
    try:
        n1, dt1 = _time_oracle(oracle, host, w, seconds)
    finally:
        oracle.set_threads(cores)
    return {"value": n * nodes / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} passes over one {w.name} batch (B={w.B}, all algorithms), {dt:.1f} s of wall time; "
                      "the checker evaluates only the nodes the walk reaches",
            "one_thread": {"value": n1 * nodes / dt1, "unit": UNIT, "cores": 1,
                           "sample": f"{n1} passes over the same batch on one thread, {dt1:.1f} s of wall time"}}


def run_reference(args):
    """The CPU checker as the reference arm: rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    from paper_2602_16994_b200 import synth
    oracle.build()
    w = synth.WORKLOADS[args.workload]
    host = synth.make_batch(w, seed=0, device="cpu").numpy()
    steps = max(1, min(args.steps, 50))
    warm = max(1, min(args.warmup, 3))
    for _ in range(warm):
        oracle_step(oracle, host, w)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(oracle, host, w)
    dt = time.perf_counter() - t0
    nodes = w.draft_nodes() * len(w.algorithms)
    value = nodes * steps / dt
    sample = f"each step = the CPU checker on one full {w.name} batch (B={w.B}), all algorithms"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "V": w.V, "algorithms": list(w.algorithms)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2602_16994_b200 import binding, shard, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the verification path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.load_library()

    w = synth.WORKLOADS[args.workload]
    bytes_per_call = w.logit_bytes()
    copies = max(2, min(24, -(-ROTATE_BYTES // bytes_per_call))) if bytes_per_call < ROTATE_BYTES else 1
    seeds = shard.rank_seeds(rank, world, copies)
    # drawn by torch's CPU generator unless asked otherwise: a seed then names the same batch on every
    # machine, and seed 0 (rank 0's first copy) is the batch the CPU checker legs run on
    if args.gen == "cpu":
        batches = [synth.make_batch(w, seed=s, device="cpu").to(dev) for s in seeds]
    else:
        batches = [synth.make_batch(w, seed=s, device=dev) for s in seeds]
    outs = binding.alloc_outputs(w.B, w.N, w.V, dev, features=w.features)
    stream = torch.cuda.current_stream()
    # arguments marshalled once per (algorithm, input copy); a call is then one C-ABI call
    prepared = {a: [binding.PreparedVerify(a, b.target_logits, b.draft_logits, b.parent, b.token, b.u_accept,
                                           b.u_bonus, w.temperature, w.top_k, w.top_p, outputs=outs)
                    for b in batches] for a in w.algorithms}
    counter = [0]
    for a in w.algorithms:               # first calls set kernel attributes: they must not fall inside a capture
        for p in prepared[a]:
            p.launch(stream)
    stat_prepared = prepared[w.algorithms[0]]
    for p in stat_prepared:
        p.launch_statistics_only(stream)
    torch.cuda.synchronize()
    launches_per_step = None
    if args.no_graph:
        def call(algo):
            p = prepared[algo][counter[0] % len(batches)]
            counter[0] += 1
            p.launch(stream)

        def step():
            for algo in w.algorithms:
                call(algo)

        def run_stats(n):
            for i in range(n):
                stat_prepared[i % len(batches)].launch_statistics_only(stream)
    else:
        # the library neither allocates nor synchronises, so a call can be captured: one graph per input
        # copy for the whole step, one per (algorithm, copy) for the per-algorithm figures
        side = torch.cuda.Stream()

        def capture(algos, copies_, stats_only=False):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for i in copies_:
                        if stats_only:
                            stat_prepared[i].launch_statistics_only(side)
                        for a in algos:
                            prepared[a][i].launch(side)
            return g

        every = list(range(len(batches)))
        before = binding.kernel_launches()
        step_graphs = [capture(w.algorithms, [i]) for i in every]
        launches_per_step = (binding.kernel_launches() - before) // len(batches)
        # a round over all input copies as one graph: consecutive steps then follow each other on the
        # device without a host launch in between
        round_graph = capture(w.algorithms, every)
        algo_round = {a: capture([a], every) for a in w.algorithms}
        algo_single = {a: [capture([a], [i]) for i in every] for a in w.algorithms}
        stat_round = capture([], every, stats_only=True)
        stat_single = [capture([], [i], stats_only=True) for i in every]

        def run_steps(n):
            for _ in range(n // len(batches)):
                round_graph.replay()
            for i in range(n % len(batches)):
                step_graphs[i].replay()

        def run_calls(algo, n):
            for _ in range(n // len(batches)):
                algo_round[algo].replay()
            for i in range(n % len(batches)):
                algo_single[algo][i].replay()

        def run_stats(n):
            for _ in range(n // len(batches)):
                stat_round.replay()
            for i in range(n % len(batches)):
                stat_single[i].replay()

    if args.no_graph:
        def run_steps(n):
            for _ in range(n):
                step()

        def run_calls(algo, n):
            for _ in range(n):
                call(algo)

    def timed_blocks(run, n, repeats):
        """``repeats`` blocks of ``n`` units each, timed on the device (barrier + synchronise on both sides of
        every block, slowest rank counted): milliseconds per unit of every block."""
        out = []
        for _ in range(repeats):
            shard.barrier(world)
            torch.cuda.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            run(n)
            t1.record(stream)
            torch.cuda.synchronize()
            shard.barrier(world)
            out.append(shard.max_over_ranks(t0.elapsed_time(t1), world, dev) / n)
        return out

    def spread(ms_list, scale=1.0):
        return {"median": statistics.median(ms_list) * scale, "min": min(ms_list) * scale,
                "max": max(ms_list) * scale, "blocks": len(ms_list)}

    R = max(1, args.repeats)
    run_steps(max(3, args.warmup))
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = binding.kernel_launches()
    step_ms = timed_blocks(run_steps, args.steps, R)
    # counted by the library at every launch site (for graphs: at capture, times the replays); per block
    gpu_launches = ((binding.kernel_launches() - launches0) // R if launches_per_step is None
                    else launches_per_step * args.steps)
    # per-algorithm call duration (the node kernel dominates a call), same rotation of cold inputs
    per_algo = {}
    for algo in w.algorithms:
        run_calls(algo, max(3, len(batches)))
        ms = timed_blocks(lambda n: run_calls(algo, n), args.steps, R)
        med = statistics.median(ms)
        per_algo[algo] = {"us_per_call": med * 1e3, "us_min": min(ms) * 1e3, "us_max": max(ms) * 1e3,
                          "gbs": bytes_per_call / med / 1e6, "nodes_per_s": w.draft_nodes() / med * 1e3}
    # the row statistics kernel by itself, same rotation of cold inputs
    run_stats(max(3, len(batches)))
    stat_ms = timed_blocks(run_stats, args.steps, R)
    # the same calls on ONE input copy, read again and again: whatever of it fits in L2 comes from there
    l2_warm = None
    if copies > 1:
        l2_warm = {}
        for algo in w.algorithms:
            if args.no_graph:
                one = lambda n, a=algo: [prepared[a][0].launch(stream) for _ in range(n)]
            else:
                one = lambda n, a=algo: [algo_single[a][0].replay() for _ in range(n)]
            one(3)
            l2_warm[algo] = spread(timed_blocks(one, args.steps, max(3, R // 3)), 1e3)["median"]
        one = ((lambda n: [stat_prepared[0].launch_statistics_only(stream) for _ in range(n)]) if args.no_graph
               else (lambda n: [stat_single[0].replay() for _ in range(n)]))
        one(3)
        l2_warm["statistics_kernel"] = spread(timed_blocks(one, args.steps, max(3, R // 3)), 1e3)["median"]
        l2_warm["unit"] = "us per call, one input copy re-read (it fits in L2): NOT an HBM figure"
    clocks = sampler.stop() if rank == 0 else None
    status_ok = bool((outs.status == 0).all().item())

    # end to end through the host-buffer entry point: pinned host inputs, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        hv = {a: binding.HostVerifier(w.B, w.N, w.V, batches[0].target_logits.dtype, dev, algorithm=a)
              for a in w.algorithms}
        hb = batches[0]
        pin = lambda t: t.cpu().pin_memory()
        host = [pin(hb.target_logits), pin(hb.draft_logits), pin(hb.parent), pin(hb.token), pin(hb.u_accept),
                pin(hb.u_bonus)]
        n_e2e = max(3, min(args.steps, 20))
        for a in w.algorithms:
            hv[a].run(*host, w.temperature, w.top_k, w.top_p)
        shard.barrier(world)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            for a in w.algorithms:
                hv[a].run(*host, w.temperature, w.top_k, w.top_p)
        dt_ms = (time.perf_counter() - t0) * 1e3
        shard.barrier(world)
        dt_ms = shard.max_over_ranks(dt_ms, world, dev)
        first = hv[w.algorithms[0]]
        e2e = {"value": world * w.draft_nodes() * len(w.algorithms) * n_e2e / dt_ms * 1e3, "unit": UNIT,
               "h2d_bytes_per_step": first.h2d_bytes() * len(w.algorithms),
               "d2h_bytes_per_step": first.d2h_bytes() * len(w.algorithms),
               "ms_per_step": dt_ms / n_e2e, "steps": n_e2e,
               "api": "spec_verify_host (C ABI, pinned host buffers in, host results out, one sync per call)"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak, peak_src = 6650.0, "fallback"
    trunc = (0 < w.top_k < w.V) or w.top_p < 1.0
    stat_med = statistics.median(stat_ms)
    achieved = bytes_per_call / stat_med / 1e6
    ms_per_step = statistics.median(step_ms)
    nodes_per_step = w.draft_nodes() * len(w.algorithms)
    line = {
        "metric": METRIC, "value": world * nodes_per_step / ms_per_step * 1e3, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
        "ms_per_step_spread": spread(step_ms), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "B_per_gpu": w.B, "N": w.N, "V": w.V, "logits": w.dtype,
                   "tree": f"delayed K={w.K} L1={w.L1} L2={w.L2}", "temperature": w.temperature, "top_k": w.top_k,
                   "top_p": w.top_p, "step": "+".join(w.algorithms) + " on one batch",
                   "launch": "host enqueue per call" if args.no_graph else
                             f"CUDA graph replay: one graph holds a round of {len(batches)} steps (one per input copy), "
                             "single-step graphs for the remainder",
                   "timing": f"{R} blocks of {args.steps} steps, each between two CUDA events on the launching stream; "
                             "the median block is reported",
                   "inputs": f"seeded, drawn on the {args.gen}",
                   "node_verifications_per_step": nodes_per_step, "logit_bytes_per_call": bytes_per_call,
                   "l2": f"{copies} input copies rotated ({copies * bytes_per_call / 1e6:.0f} MB touched between "
                         f"reuses, L2 is {L2_BYTES / 1e6:.0f} MB)" if copies > 1 else "inputs larger than L2"},
        "hbm_gbs": world * bytes_per_call * len(w.algorithms) / ms_per_step / 1e6,
        "per_algorithm": per_algo,
        # the kernel that reads the logits from HBM, timed by itself; the fractions of whole calls (its
        # bytes over the duration of statistics + node kernel) are given beside it
        "roofline": {"bound": "hbm", "kernel": STAT_KERNEL[trunc], "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                     "kernel_us": spread(stat_ms, 1e3),
                     "frac_of_8TBs_nominal": achieved / 8000.0,
                     "traffic": None if trunc else TRAFFIC_BYTES.get(w.name),
                     "algorithmic_bytes_per_launch": bytes_per_call,
                     "whole_call_frac": {a: per_algo[a]["gbs"] / peak for a in w.algorithms},
                     "whole_call_traffic": None if trunc else TRAFFIC_CALL_BYTES.get(w.name)},
        "l2_warm_us": l2_warm,
        "clocks": clocks, "gpu_launches": gpu_launches,
        "status_ok": status_ok,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, args.cpu_seconds)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
