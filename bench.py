"""Benchmark of batched draft-tree verification (SpecInfer + Traversal Verification) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole verification path over one batch of synthetic draft trees: every
algorithm the workload lists (SpecInfer, Traversal Verification) is run once on the batch through
the C-ABI library, logits already resident in HBM.  Consecutive calls use different input copies so
that more than the L2 capacity is touched before a copy is read again (reads come from HBM).
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
# kernels of one call; the roofline figure is taken over the whole call (all of its kernels), so it
# understates the fraction the streaming kernel reaches on its own
KERNELS = {"specinfer": "spec_row_partial_kernel + spec_walk_kernel (whole specinfer call)",
           "traversal": "spec_row_partial_kernel + spec_tree_kernel (whole traversal call)"}
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (cold L2), for the kernels of a SpecInfer call on the headline workload: the row statistics
# kernel (69.80 + 0.76 MB: every logit once) and the walk kernel (4.08 MB: the rows of the resident
# nodes, which come from L2 in the benchmark).  Other workloads: not captured.
TRAFFIC_BYTES = {"cfg2_llama3_b8": 69_798_912 + 760_320 + 4_075_776}


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


def cpu_baseline(w, seconds: float) -> dict:
    import oracle
    from paper_2602_16994_b200 import synth
    oracle.build()
    host = synth.make_batch(w, seed=0, device="cpu").numpy()
    oracle_step(oracle, host, w)                       # warm-up (page-in, thread pool)
    n, t0 = 0, time.perf_counter()
    while True:
        oracle_step(oracle, host, w)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or n >= 10000:
            break
    nodes = n * w.draft_nodes() * len(w.algorithms)
    return {"value": nodes / dt, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "sample": f"{n} passes over one {w.name} batch (B={w.B}, all algorithms), {dt:.1f} s of wall time; "
                      "the checker evaluates only the nodes the walk reaches"}


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
    else:
        # the library neither allocates nor synchronises, so a call can be captured: one graph per input
        # copy for the whole step, one per (algorithm, copy) for the per-algorithm figures
        side = torch.cuda.Stream()

        def capture(algos, copies_):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for i in copies_:
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

    if args.no_graph:
        def run_steps(n):
            for _ in range(n):
                step()

        def run_calls(algo, n):
            for _ in range(n):
                call(algo)

    run_steps(max(3, args.warmup))
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    shard.barrier(world)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = binding.kernel_launches()
    e0.record(stream)
    run_steps(args.steps)
    e1.record(stream)
    torch.cuda.synchronize()
    # counted by the library at every launch site (for graphs: at capture, times the replays)
    gpu_launches = (binding.kernel_launches() - launches0) if launches_per_step is None else launches_per_step * args.steps
    shard.barrier(world)
    ms_total = shard.max_over_ranks(e0.elapsed_time(e1), world, dev)
    # per-algorithm call duration (the node kernel dominates a call), same rotation of cold inputs
    per_algo = {}
    for algo in w.algorithms:
        run_calls(algo, max(3, len(batches)))
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        run_calls(algo, args.steps)
        a1.record(stream)
        torch.cuda.synchronize()
        ms = a0.elapsed_time(a1) / args.steps
        per_algo[algo] = {"us_per_call": ms * 1e3, "gbs": bytes_per_call / ms / 1e6,
                          "nodes_per_s": w.draft_nodes() / ms * 1e3}
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
    dom = w.algorithms[0]
    achieved = per_algo[dom]["gbs"]
    ms_per_step = ms_total / args.steps
    nodes_per_step = w.draft_nodes() * len(w.algorithms)
    line = {
        "metric": METRIC, "value": world * nodes_per_step / ms_per_step * 1e3, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "B_per_gpu": w.B, "N": w.N, "V": w.V, "logits": w.dtype,
                   "tree": f"delayed K={w.K} L1={w.L1} L2={w.L2}", "temperature": w.temperature, "top_k": w.top_k,
                   "top_p": w.top_p, "step": "+".join(w.algorithms) + " on one batch",
                   "launch": "host enqueue per call" if args.no_graph else
                             f"CUDA graph replay: one graph holds a round of {len(batches)} steps (one per input copy), "
                             "single-step graphs for the remainder",
                   "node_verifications_per_step": nodes_per_step, "logit_bytes_per_call": bytes_per_call,
                   "l2": f"{copies} input copies rotated ({copies * bytes_per_call / 1e6:.0f} MB touched between "
                         f"reuses, L2 is {L2_BYTES / 1e6:.0f} MB)" if copies > 1 else "inputs larger than L2"},
        "hbm_gbs": world * bytes_per_call * len(w.algorithms) / ms_per_step / 1e6,
        "per_algorithm": per_algo,
        "roofline": {"bound": "hbm", "kernel": KERNELS[dom], "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                     "frac_of_8TBs_nominal": achieved / 8000.0, "traffic": TRAFFIC_BYTES.get(w.name),
                     "algorithmic_bytes_per_launch": bytes_per_call},
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
