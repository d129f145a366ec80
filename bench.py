"""Benchmark of the BPDQ weight-only linear layer (decode GEMV, prefill GEMM, dequant) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]
    python bench.py --case few --out 29568 --in 8192 --K 2 --M 16 --iters 3      (one kernel on one linear, for profilers)

One JSON line on stdout.  The headline workload is a Qwen2.5-72B-shaped decoder layer at K = 2
bit-planes, group 128, one token (M = 1): a step is one pass of bpdq_linear over the layer's seven
linears.  Several distinct copies of the layer are rotated between steps so that no weight byte can
be served from L2.  The timed region is `--steps` steps between two barriers; it is repeated
TIMED_BLOCKS times back to back (one barrier before the first and one after the last block, an event
between blocks) and the median block is reported: a block of 20 steps lasts about a millisecond, and
the first launches after a pause run slower than the steady state.  `value` is the useful HBM bytes (packed planes + coefficients + x + y) moved per
second; the `roofline` object relates it to the measured copy bandwidth.  Further timed sections
(K = 3 layer, fused qkv / gate-up handles, prefill GEMM, dequant) are reported under `sections`.

With --gpus N > 1 (launched under torchrun) every rank runs an independent replica of the same
workload ("replicas only": the path has no exchange step); the value is the sum over ranks divided
by the slowest rank's time.

--impl reference times the plain C++ checker under oracle/ on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_04163_b200 import synth  # noqa: E402

METRIC = "bpdq_gemv_useful_hbm_gbs_batch1_72b_layer"
UNIT = "GB/s"
GROUP = 128
HBM_NOMINAL_GBS = 8000.0
FALLBACK_HBM_GBS, FALLBACK_TFLOPS = 6650.0, 1590.0
# dram__bytes_read.sum + dram__bytes_write.sum of the headline launch, from the ncu capture summarised in
# profiles/gemv_lut_K2_layer72b_batch_M1.md (set to None whenever the kernel changes until the counters are taken again)
GEMV_TRAFFIC_BYTES_PER_LAUNCH = 264_899_840
# the same for one launch of the 512-token tcgen05 kernel on the gate projection at K = 3, M = 2048
# (profiles/gemm_wide_K3_gate_29568x8192_M2048.md); the prefill sections time whole layers, so this is context for them
GEMM_GATE_K3_M2048_TRAFFIC_BYTES = 553_668_096
TIMED_BLOCKS = 25


def useful_bytes(out: int, in_: int, K: int, g: int, M: int) -> int:
    """Algorithmic HBM bytes of one linear call: packed planes + binary16 coefficients + x + y."""
    return out * in_ * K // 8 + out * (-(-in_ // g)) * (K + 1) * 2 + M * in_ * 2 + M * out * 2    # ceil(in / g) groups: a last one may be short


def layer_bytes(shapes, K: int, M: int) -> int:
    return sum(useful_bytes(o, i, K, GROUP, M) for _, o, i in shapes)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "tflops": float(d["bf16_tflops"]),
                "tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "tflops": FALLBACK_TFLOPS, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for t, r in self.rows if t0 <= t <= t1 + 0.2 and len(r) >= 7] or [r for _, r in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names) if any(r[3 + k].lower().startswith("active") for r in rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][1]), "reasons": reasons,
                "samples": len(rows), "power_w_max": max(float(r[2]) for r in rows)}


# ------------------------------------------------------------------------------------------------
# reference arm: the checker under oracle/, as it stands, on the host cores
# ------------------------------------------------------------------------------------------------
def oracle_sample(shapes, K: int, rows_per_linear: int, seed: int = 0):
    """Logical tensors of `rows_per_linear` evenly spaced output rows of every linear of the layer."""
    sample = []
    for li, (name, out, in_) in enumerate(shapes):
        s = synth.linear_seed(seed, 0, li, K)
        rows = np.unique(np.linspace(0, out - 1, rows_per_linear).astype(np.int64))
        sample.append((name, out, in_, synth.plane_bits(s, out, in_, K, rows),
                       synth.coefficients(s, out, in_, K, GROUP, rows), synth.activations(s + 1, 1, in_)))
    return sample


def time_oracle(sample, K: int):
    """Runs the checker's linear map over the sample once; returns (seconds, useful bytes covered)."""
    import oracle
    covered = 0
    t0 = time.perf_counter()
    for _, out, in_, bits, coef, x in sample:
        oracle.linear(bits, coef, x, GROUP)
        n = bits.shape[1]
        covered += useful_bytes(n, in_, K, GROUP, 1)
    return time.perf_counter() - t0, covered


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def time_oracle_threads(sample, K: int, threads: int, M: int = 1):
    """The unchanged checker function on `threads` host threads, each on its own slice of the sample's output rows
    (the foreign call releases the interpreter lock); returns (seconds, useful bytes covered, weights covered)."""
    import concurrent.futures
    import oracle
    jobs = []
    for _, out, in_, bits, coef, x in sample:
        n = bits.shape[1]
        cuts = np.linspace(0, n, min(threads, n) + 1).astype(int)
        for a, b in zip(cuts[:-1], cuts[1:]):
            if b > a:
                jobs.append((np.ascontiguousarray(bits[:, a:b]), np.ascontiguousarray(coef[:, a:b]), x))
    covered = sum(useful_bytes(b.shape[1], i, K, GROUP, M) for _, _, i, b, _, _ in sample)
    weights = sum(b.shape[1] * i for _, _, i, b, _, _ in sample)
    t0 = time.perf_counter()
    with concurrent.futures.ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda j: oracle.linear(j[0], j[1], j[2], GROUP), jobs))
    return time.perf_counter() - t0, covered, weights


def run_reference(args, rank: int):
    if rank != 0:
        return
    shapes, K = synth.QWEN25_72B_LAYER, 2
    # bounded sample: the whole run (warm-up included) stays near one minute at the checker's ~8e6 weights/s
    cols = sum(i for _, _, i in shapes)
    rows = max(2, min(4096, int(60.0 * 8e6 * host_cores() / (cols * max(1, args.steps + args.warmup)))))
    sample = oracle_sample(shapes, K, rows)
    import oracle
    oracle.build()
    cores = host_cores()
    for _ in range(args.warmup):
        time_oracle_threads(sample, K, cores)
    t_total, covered = 0.0, 0
    for _ in range(args.steps):
        dt, nb, _ = time_oracle_threads(sample, K, cores)
        t_total += dt
        covered += nb
    value = covered / t_total / 1e9
    desc = f"{rows} evenly spaced output rows of each of the 7 linears per step, rows split over {cores} host threads"
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "qwen2.5-72b-shaped decoder layer, K=2, g=128, M=1 (7 linears)", "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------
def slowest_rank(times_ms, world: int, device: str):
    """Max over ranks of each timing (the job is as slow as its slowest replica); identity for one rank."""
    import torch
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def replica_throughput_gbs(bytes_per_step: int, steps: int, world: int, ms_slowest: float) -> float:
    """Whole-job rate of `world` independent replicas: all their bytes over the slowest rank's time."""
    return world * bytes_per_step * steps / (ms_slowest * 1e-3) / 1e9


class Layer:
    """Handles of one decoder layer's linears, generated on the device from a seed."""

    def __init__(self, shapes, K: int, seed: int, layer: int, max_M: int):
        from paper_2602_04163_b200 import binding
        self.handles = []
        for li, (name, out, in_) in enumerate(shapes):
            self.handles.append((name, binding.Handle(out, in_, K, GROUP, None, synth.linear_seed(seed, layer, li, K), max_M)))

    def destroy(self):
        for _, h in self.handles:
            h.bpdq_destroy()


def graph_replay_ms(torch, binding, stream, layers, groups, xs, ys, n):
    """Records the batched launches of every layer copy (M = 1) into one CUDA graph and times n layers' worth of replays."""
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for hs in layers:
            for grp in groups:
                binding.bpdq_linear_batch([hs[j] for j in grp], [xs[hs[j].in_].data_ptr() for j in grp], [ys[j].data_ptr() for j in grp],
                                          1, side.cuda_stream)
    replays = max(1, n // len(layers))

    def run():
        for _ in range(replays):
            graph.replay()
    run()
    return event_time_ms(torch, run, stream) * n / (replays * len(layers))


def event_time_ms(torch, fn, stream):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    fn()
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1)


def run_cuda(args, rank: int, world: int, local_rank: int):
    import torch
    import torch.distributed as dist
    from paper_2602_04163_b200 import binding

    binding.lib()                      # raises if the CUDA library is missing: there is no other path
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    peaks = measured_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    shapes, K, M = synth.QWEN25_72B_LAYER, 2, 1
    copies = 4
    layers = [Layer(shapes, K, 0, c, 1) for c in range(copies)]
    xs = {in_: torch.from_numpy(synth.activations(7, 1, in_).view(np.int16).copy()).cuda().view(torch.float16)
          for in_ in sorted({i for _, _, i in shapes})}
    ys = {out: torch.empty((1, out), dtype=torch.float16, device="cuda") for out in sorted({o for _, o, _ in shapes})}
    ys_each = [torch.empty((1, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes]
    x_ptrs = [xs[i].data_ptr() for _, _, i in shapes]
    y_ptrs = [y.data_ptr() for y in ys_each]

    def step(layer):
        # the layer's seven linears have independent inputs in this workload: one launch covers them all
        binding.bpdq_linear_batch([h for _, h in layer.handles], x_ptrs, y_ptrs, M, sp)

    def step_separate(layer):
        for k, (name, h) in enumerate(layer.handles):
            h.bpdq_linear(x_ptrs[k], y_ptrs[k], M, sp)

    launches0 = sum(h.bpdq_launch_count() for L in layers for _, h in L.handles)
    for w in range(args.warmup):
        step(layers[w % copies])
    barrier()
    launches1 = sum(h.bpdq_launch_count() for L in layers for _, h in L.handles)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    t_wall0 = time.time()
    # the timed region: TIMED_BLOCKS blocks of exactly `steps` steps, back to back between two barriers, an event on the
    # launching stream between blocks; the median block is the one reported
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(TIMED_BLOCKS + 1)]
    barrier()
    marks[0].record(stream)
    for blk in range(TIMED_BLOCKS):                                 # back to back: no host wait between blocks
        for s in range(args.steps):
            step(layers[(blk * args.steps + s) % copies])
        marks[blk + 1].record(stream)
    barrier()
    block_ms = [marks[b].elapsed_time(marks[b + 1]) for b in range(TIMED_BLOCKS)]
    ms_first = block_ms[0]
    ms_total = sorted(block_ms)[len(block_ms) // 2]
    t_wall1 = time.time()
    launches2 = sum(h.bpdq_launch_count() for L in layers for _, h in L.handles)

    # the timed region is microseconds long at small step counts; keep the GPU under the same load a
    # little longer so that nvidia-smi (100 ms period) sees the clocks it ran at
    t_hold = time.time()
    while time.time() - t_hold < 1.0:
        for s in range(50):
            step(layers[s % copies])
        torch.cuda.synchronize()
    clocks = sampler.stop(t_wall0, time.time())

    # end to end: x in pinned host memory, y back to pinned host memory, every step, through the C ABI
    xh = {in_: torch.from_numpy(synth.activations(7, 1, in_).view(np.int16).copy()).view(torch.float16).pin_memory()
          for in_ in xs}
    yh = {out: torch.empty((1, out), dtype=torch.float16).pin_memory() for out in ys}

    yh_each = [torch.empty((1, o), dtype=torch.float16).pin_memory() for _, o, _ in shapes]
    xh_ptrs = [xh[i].data_ptr() for _, _, i in shapes]
    yh_ptrs = [y.data_ptr() for y in yh_each]

    def step_host(layer):
        binding.bpdq_linear_batch_host([h for _, h in layer.handles], xh_ptrs, yh_ptrs, M, sp)

    for w in range(max(3, args.warmup)):
        step_host(layers[w % copies])
    barrier()
    t0 = time.perf_counter()
    for s in range(args.steps):
        step_host(layers[s % copies])
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    ms_total, e2e_ms = slowest_rank([ms_total, e2e_s * 1e3], world, "cuda")
    bytes_step = layer_bytes(shapes, K, M)
    value = replica_throughput_gbs(bytes_step, args.steps, world, ms_total)
    e2e_value = replica_throughput_gbs(bytes_step, args.steps, world, e2e_ms)
    per_gpu = value / world
    n_launch = (launches2 - launches1) // TIMED_BLOCKS              # kernels launched inside one timed block

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": "qwen2.5-72b-shaped decoder layer, K=2, g=128, M=1 (7 linears: q k v o gate up down, each with its own x, "
                                   "issued as one bpdq_linear_batch call; sections.seven_separate_calls times seven bpdq_linear calls)",
                       "l2": f"inputs larger than L2: {copies} distinct layer copies of {bytes_step / 1e6:.1f} MB rotated between steps",
                       "useful_bytes_per_step": bytes_step, "parallelism": "replicas only" if world > 1 else "single GPU",
                       "timing": f"median of {TIMED_BLOCKS} back-to-back blocks of `steps` steps between two barriers; first block {ms_first / args.steps * 1e3:.1f} us per step"},
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": sum(2 * M * i for _, _, i in shapes), "d2h_bytes_per_step": sum(2 * M * o for _, o, _ in shapes),
                    "path": "bpdq_linear_batch_host, every step: one gather launch reads the seven x from pinned host memory, the kernel "
                            "stores the seven y into pinned host memory, one stream wait"},
            "gpu_launches": n_launch, "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "gemv_lut_kernel", "achieved": per_gpu, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": per_gpu / peaks["hbm_gbs"], "peak_source": peaks["source"],
                         "frac_of_nominal_8tbs": per_gpu / HBM_NOMINAL_GBS, "traffic": GEMV_TRAFFIC_BYTES_PER_LAUNCH,
                         "launches_per_step": 1, "algorithmic_bytes_per_launch": bytes_step}}

    # the same layer as seven separate bpdq_linear calls
    for w in range(3):
        step_separate(layers[w % copies])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s_ in range(args.steps):
        step_separate(layers[s_ % copies])
    e1.record(stream)
    e1.synchronize()
    ms_sep = e0.elapsed_time(e1) / args.steps
    separate = {"launches_per_layer": len(shapes), "us_per_layer": ms_sep * 1e3, "gbs": bytes_step / (ms_sep * 1e-3) / 1e9,
                "frac_measured": bytes_step / (ms_sep * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    if rank == 0 and not args.no_extras:
        line["sections"] = extra_sections(torch, binding, args, peaks, sp, stream)
        line["sections"]["seven_separate_calls"] = separate
        line["sections"]["decode_sweep_80_layers_K2"] = full_stack_section(torch, binding, peaks, sp, stream)
        # the paper's headline deployment format (W2-G256 on the 72B model) as a whole stack
        line["sections"]["decode_sweep_80_layers_W2-G256"] = full_stack_section(torch, binding, peaks, sp, stream, group=256)
        dg = line["sections"].get("gemv_layer_batched_decoder_groups_K2", {})
        line["config"]["same_layer_other_issue_orders"] = {
            "decoder_legal_groups_qkv_o_gateup_down": {"us_per_layer": dg.get("us_per_layer"), "frac_measured": dg.get("frac_measured")},
            "seven_bpdq_linear_calls": {"us_per_layer": separate["us_per_layer"], "frac_measured": separate["frac_measured"]}}
    for L in layers:
        L.destroy()

    if rank == 0:
        if world == 1:
            line["cpu_baseline"] = cpu_baseline(shapes, K)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def cpu_baseline(shapes, K):
    """The checker as it stands on the machine's host cores, on bounded samples of the benchmark's workloads (about 25 s):
    the decode layer on every core (row-parallel wrapper around the unchanged function) and on one core, and a
    subset of the prefill layer whose full-size time is extrapolated from it."""
    import oracle
    oracle.build()
    cores = host_cores()
    rows1 = 2304
    dt1, cov1, _ = time_oracle_threads(oracle_sample(shapes, K, rows1), K, 1)
    rows_all = min(29568, 2560 * cores)
    dta, cova, _ = time_oracle_threads(oracle_sample(shapes, K, rows_all), K, cores)
    # prefill subset: 16 tokens through `rows_p` rows of every linear at K = 3; the checker's cost per (weight, token)
    # pair is taken from it and scaled to 8192 tokens x all rows (decode cost per weight is paid once per row)
    Kp, Mp, rows_p = 3, 16, 96 * cores
    samp = []
    for li, (name, out, in_) in enumerate(shapes):
        sd = 700 + li
        rows = np.unique(np.linspace(0, out - 1, rows_p).astype(np.int64))
        samp.append((name, out, in_, synth.plane_bits(sd, out, in_, Kp, rows), synth.coefficients(sd, out, in_, Kp, GROUP, rows),
                     synth.activations(3, 8192, in_, tokens=np.arange(Mp))))
    dtp, _, wp = time_oracle_threads(samp, Kp, cores, Mp)
    full_weights = sum(o * i for _, o, i in shapes)
    est_s_8192 = dtp / (wp * Mp) * full_weights * 8192          # upper bound: charges the per-weight decode to every token
    flops_8192 = 2.0 * 8192 * full_weights
    return {"value": cova / dta / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dta,
            "sample": f"{rows_all} evenly spaced output rows of each of the 7 linears of the layer (M=1), one pass, rows split over {cores} threads",
            "single_thread": {"value": cov1 / dt1 / 1e9, "unit": UNIT, "cores": 1, "seconds": dt1,
                              "sample": f"{rows1} evenly spaced output rows of each of the 7 linears (M=1), one pass"},
            "prefill_subset": {"K": Kp, "tokens": Mp, "rows_per_linear": rows_p, "cores": cores, "seconds": dtp,
                               "extrapolated_seconds_layer_M8192": est_s_8192,
                               "extrapolated_tflops_layer_M8192": flops_8192 / est_s_8192 / 1e12,
                               "note": "extrapolated from the subset by (weights x tokens); not measured at full size"}}


def extra_sections(torch, binding, args, peaks, sp, stream):
    """Per-linear GEMV at K=2 and K=3, fused handles, dequant and the prefill GEMM, each timed alone."""
    out = {}
    steps = max(5, min(args.steps, 20))
    l2_flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn, n=steps):
        ts = []
        for _ in range(3):
            fn()
        for _ in range(n):
            l2_flush.zero_()
            ts.append(event_time_ms(torch, fn, stream))
        ts.sort()
        return ts[len(ts) // 2], ts[0]

    shapes72 = synth.QWEN25_72B_LAYER
    per_linear = []
    cases = [("q/o", 8192, 8192), ("k/v", 1024, 8192), ("gate/up", 29568, 8192), ("down", 8192, 29568),
             ("qkv fused", 10240, 8192), ("gate+up fused", 59136, 8192)]
    for K in (2, 3):
        for name, o, i in cases:
            h = binding.Handle(o, i, K, GROUP, None, 11, 1)
            x = torch.from_numpy(synth.activations(3, 1, i).view(np.int16).copy()).cuda().view(torch.float16)
            y = torch.empty((1, o), dtype=torch.float16, device="cuda")
            med, best = timed(lambda: h.bpdq_linear(x.data_ptr(), y.data_ptr(), 1, sp))
            b = useful_bytes(o, i, K, GROUP, 1)
            per_linear.append({"linear": name, "out": o, "in": i, "K": K, "us_median": med * 1e3, "us_best": best * 1e3,
                               "gbs": b / (med * 1e-3) / 1e9, "frac_measured": b / (med * 1e-3) / 1e9 / peaks["hbm_gbs"]})
            h.bpdq_destroy()
    out["gemv_per_linear_l2_flushed"] = per_linear

    # dequant of the gate projection
    for K in (2, 3):
        o, i = 29568, 8192
        h = binding.Handle(o, i, K, GROUP, None, 12, 1)
        w = torch.empty((o, i), dtype=torch.float16, device="cuda")
        med, best = timed(lambda: h.bpdq_dequant(w.data_ptr(), sp), 5)
        b = h.packed_bytes + o * i * 2
        out[f"dequant_gate_K{K}"] = {"ms_median": med, "gbs": b / (med * 1e-3) / 1e9,
                                     "frac_measured": b / (med * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        h.bpdq_destroy()
        del w

    def xt(M, in_, seed=3):
        return torch.from_numpy(synth.activations(seed, M, in_).view(np.int16).copy()).cuda().view(torch.float16)

    # decoder layer with fused handles (q|k|v share x, gate|up share x): 4 launches instead of 7, same bytes
    for K in (2, 3):
        fused = [("qkv", 10240, 8192), ("o", 8192, 8192), ("gate_up", 59136, 8192), ("down", 8192, 29568)]
        copies = 3
        layers = [[binding.Handle(o, i, K, GROUP, None, 500 + 10 * c + li, 1) for li, (_, o, i) in enumerate(fused)] for c in range(copies)]
        xs = {8192: xt(1, 8192), 29568: xt(1, 29568)}
        ys = {o: torch.empty((1, o), dtype=torch.float16, device="cuda") for _, o, _ in fused}
        b = sum(useful_bytes(o, i, K, GROUP, 1) for _, o, i in fused)
        n = 60

        def run_layers():
            for k in range(n):
                for h in layers[k % copies]:
                    h.bpdq_linear(xs[h.in_].data_ptr(), ys[h.out].data_ptr(), 1, sp)
        run_layers()
        ms = event_time_ms(torch, run_layers, stream) / n
        out[f"gemv_layer_fused_handles_K{K}"] = {"launches_per_layer": 4, "us_per_layer": ms * 1e3, "gbs": b / (ms * 1e-3) / 1e9,
                                                 "frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                                 "l2": f"{copies} layer copies of {b / 1e6:.0f} MB rotated"}
        for L in layers:
            for h in L:
                h.bpdq_destroy()

    # the same layer through bpdq_linear_batch: one launch for all seven linears (legitimate when, as in this
    # benchmark, every linear has its own input), and the grouping a decoder allows: {q,k,v} {o} {gate,up} {down}
    for K in (2, 3):
        shapes7 = synth.QWEN25_72B_LAYER
        copies = 3
        layers = [[binding.Handle(o, i, K, GROUP, None, 800 + 10 * c + li, 1) for li, (_, o, i) in enumerate(shapes7)] for c in range(copies)]
        xs = {8192: xt(1, 8192), 29568: xt(1, 29568)}
        ys = [torch.empty((1, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes7]
        b = layer_bytes(shapes7, K, 1)
        n = 60
        for label, groups in (("one_launch", [[0, 1, 2, 3, 4, 5, 6]]), ("decoder_groups", [[0, 1, 2], [3], [4, 5], [6]])):
            def run_batched():
                for k in range(n):
                    hs = layers[k % copies]
                    for grp in groups:
                        binding.bpdq_linear_batch([hs[j] for j in grp], [xs[hs[j].in_].data_ptr() for j in grp],
                                                  [ys[j].data_ptr() for j in grp], 1, sp)
            run_batched()
            ms = event_time_ms(torch, run_batched, stream) / n
            out[f"gemv_layer_batched_{label}_K{K}"] = {"launches_per_layer": len(groups), "us_per_layer": ms * 1e3,
                                                       "gbs": b / (ms * 1e-3) / 1e9, "frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                                       "l2": f"{copies} layer copies of {b / 1e6:.0f} MB rotated"}
            if label == "decoder_groups":
                # the same launches recorded once into a CUDA graph (all copies, so that the rotation stays) and replayed
                ms_g = graph_replay_ms(torch, binding, stream, layers, groups, xs, ys, n) / n
                out[f"gemv_layer_batched_{label}_K{K}"]["cuda_graph_us_per_layer"] = ms_g * 1e3
        for L in layers:
            for h in L:
                h.bpdq_destroy()

    # Qwen2.5-7B-shaped layer (69 MB packed at K = 2: five copies rotated to stay out of L2), one batched launch
    for K in (2, 3):
        shapes7b = synth.QWEN25_7B_LAYER
        copies = 5
        layers = [[binding.Handle(o, i, K, GROUP, None, 900 + 10 * c + li, 1) for li, (_, o, i) in enumerate(shapes7b)] for c in range(copies)]
        xs = {i: xt(1, i) for i in sorted({i for _, _, i in shapes7b})}
        ys = [torch.empty((1, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes7b]
        b = layer_bytes(shapes7b, K, 1)
        n = 100

        def run_7b():
            for k in range(n):
                hs = layers[k % copies]
                binding.bpdq_linear_batch(hs, [xs[h.in_].data_ptr() for h in hs], [y.data_ptr() for y in ys], 1, sp)
        run_7b()
        ms = event_time_ms(torch, run_7b, stream) / n
        out[f"gemv_layer_7b_batched_K{K}"] = {"launches_per_layer": 1, "us_per_layer": ms * 1e3, "gbs": b / (ms * 1e-3) / 1e9,
                                              "frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                              "l2": f"{copies} layer copies of {b / 1e6:.0f} MB rotated"}
        # the grouping a decoder allows, as direct calls and as a replayed CUDA graph (small launches: here the host's
        # launch cost shows)
        groups7b = [[0, 1, 2], [3], [4, 5], [6]]

        def run_7b_groups():
            for k in range(n):
                hs = layers[k % copies]
                for grp in groups7b:
                    binding.bpdq_linear_batch([hs[j] for j in grp], [xs[hs[j].in_].data_ptr() for j in grp], [ys[j].data_ptr() for j in grp], 1, sp)
        run_7b_groups()
        ms_d = event_time_ms(torch, run_7b_groups, stream) / n
        ms_g = graph_replay_ms(torch, binding, stream, layers, groups7b, xs, ys, n) / n
        out[f"gemv_layer_7b_decoder_groups_K{K}"] = {"launches_per_layer": 4, "us_per_layer": ms_d * 1e3, "cuda_graph_us_per_layer": ms_g * 1e3,
                                                    "gbs": b / (ms_d * 1e-3) / 1e9, "frac_measured": b / (ms_d * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        for L in layers:
            for h in L:
                h.bpdq_destroy()

    # token-count sweep on the gate and down projections: all three kernels (the dispatch thresholds come from it) and
    # what bpdq_linear itself picks; an L2 flush before every launch
    sweep = []
    for K in (2, 3):
        for name, o, i in (("gate", 29568, 8192), ("down", 8192, 29568)):
            h = binding.Handle(o, i, K, GROUP, None, 13, 64)
            for M in (1, 2, 4, 8, 16, 32, 64):
                x = xt(M, i)
                y = torch.empty((M, o), dtype=torch.float16, device="cuda")
                rec = {"linear": name, "K": K, "M": M}
                for kname, kid in (("lut", binding.KERNEL_GEMV), ("few", binding.KERNEL_FEW), ("tensor", binding.KERNEL_GEMM)):
                    if (kid == binding.KERNEL_GEMV and M > binding.GEMV_MAX_M) or (kid == binding.KERNEL_FEW and M > binding.FEW_MAX_M):
                        continue
                    med, _ = timed(lambda: h.bpdq_linear_ex(x.data_ptr(), y.data_ptr(), M, kid, sp), 5)
                    rec[f"us_{kname}"] = med * 1e3
                best = min(v for k, v in rec.items() if k.startswith("us_"))
                rec["gbs_best"] = useful_bytes(o, i, K, GROUP, M) / (best * 1e-6) / 1e9
                rec["frac_measured_best"] = rec["gbs_best"] / peaks["hbm_gbs"]
                med, _ = timed(lambda: h.bpdq_linear(x.data_ptr(), y.data_ptr(), M, sp), 5)
                rec["us_dispatcher"] = med * 1e3
                sweep.append(rec)
            h.bpdq_destroy()
    out["token_sweep"] = sweep

    # prefill on the tensor-core kernel: one 72B-shaped layer at K = 3, M = 2048 and M = 8192
    shapes = synth.QWEN25_72B_LAYER
    for K, M in ((3, 2048), (3, 8192), (2, 8192)):
        hs = [binding.Handle(o, i, K, GROUP, None, 700 + li, M) for li, (_, o, i) in enumerate(shapes)]
        xs = {8192: xt(M, 8192), 29568: xt(M, 29568)}
        ys = {o: torch.empty((M, o), dtype=torch.float16, device="cuda") for o in sorted({o for _, o, _ in shapes})}
        flops = sum(2.0 * M * o * i for _, o, i in shapes)

        def run_prefill():
            for h in hs:
                h.bpdq_linear(xs[h.in_].data_ptr(), ys[h.out].data_ptr(), M, sp)
        run_prefill()
        ts = sorted(event_time_ms(torch, run_prefill, stream) for _ in range(3))
        ms = ts[1]
        per = []
        for (name, o, i), h in zip(shapes, hs):
            if name in ("gate", "down", "q"):
                t1 = sorted(event_time_ms(torch, lambda: h.bpdq_linear(xs[i].data_ptr(), ys[o].data_ptr(), M, sp), stream) for _ in range(3))[1]
                per.append({"linear": name, "ms": t1, "tflops": 2.0 * M * o * i / (t1 * 1e-3) / 1e12})
        tf = flops / (ms * 1e-3) / 1e12
        out[f"prefill_gemm_layer_K{K}_M{M}"] = {
            "ms_per_layer": ms, "tflops": tf, "per_linear": per,
            "roofline": {"bound": "tensor", "kernel": "gemm_wide_kernel", "achieved": tf, "peak": peaks["tflops"], "unit": "TFLOP/s",
                         "frac": tf / peaks["tflops"], "frac_of_sustained": tf / peaks["tflops_sustained"],
                         "peak_source": peaks["source"] + " bf16 burst (fp16 has the same nominal rate)",
                         "traffic": None, "traffic_gate_launch_K3_M2048": GEMM_GATE_K3_M2048_TRAFFIC_BYTES}}
        for h in hs:
            h.bpdq_destroy()
        del xs, ys

    # the paper's own formats (Table 1) on the 72B-shaped layer: decode as one batched launch, prefill at M = 8192
    for tag, K, g in (("W2-G64", 2, 64), ("W3-G64", 3, 64), ("W2-G256", 2, 256), ("W4-G128", 4, 128)):
        copies = 3
        gof = lambda i: g                             # 29568 input columns are 115.5 groups of 256: the last group of a row is short
        layers = [[binding.Handle(o, i, K, gof(i), None, 1100 + 10 * c + li, 1) for li, (_, o, i) in enumerate(shapes)] for c in range(copies)]
        xs1 = {8192: xt(1, 8192), 29568: xt(1, 29568)}
        ys1 = [torch.empty((1, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes]
        b = sum(useful_bytes(o, i, K, gof(i), 1) for _, o, i in shapes)
        n = 60

        def run_fmt():
            for k in range(n):
                hs_ = layers[k % copies]
                binding.bpdq_linear_batch(hs_, [xs1[h.in_].data_ptr() for h in hs_], [y.data_ptr() for y in ys1], 1, sp)
        run_fmt()
        ms = event_time_ms(torch, run_fmt, stream) / n
        rec = {"K": K, "group": g, "bits_per_weight": K + 16.0 * (K + 1) / g, "decode_us_per_layer": ms * 1e3, "decode_gbs": b / (ms * 1e-3) / 1e9,
               "decode_frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        for L in layers:
            for h in L:
                h.bpdq_destroy()
        M = 8192
        hs = [binding.Handle(o, i, K, gof(i), None, 1200 + li, M) for li, (_, o, i) in enumerate(shapes)]
        xs = {8192: xt(M, 8192), 29568: xt(M, 29568)}
        ys = {o: torch.empty((M, o), dtype=torch.float16, device="cuda") for o in sorted({o for _, o, _ in shapes})}

        def run_prefill_fmt():
            for h in hs:
                h.bpdq_linear(xs[h.in_].data_ptr(), ys[h.out].data_ptr(), M, sp)
        run_prefill_fmt()
        msp = sorted(event_time_ms(torch, run_prefill_fmt, stream) for _ in range(3))[1]
        tf = sum(2.0 * M * o * i for _, o, i in shapes) / (msp * 1e-3) / 1e12
        rec.update({"prefill_M8192_ms_per_layer": msp, "prefill_tflops": tf, "prefill_frac_measured_burst": tf / peaks["tflops"]})
        out[f"paper_format_{tag}"] = rec
        for h in hs:
            h.bpdq_destroy()
        del xs, ys

    # steps around the linears: input-channel permutation and bias on the gate projection (M = 1 and M = 8192), the
    # gated unit over (gate, up) as one call, and planes made by the data-free producer instead of random ones
    for K in (2,):
        o, i = 29568, 8192
        hs3 = [binding.Handle(o, i, K, GROUP, None, 1400 + c, 8192) for c in range(3)]
        rec = {}
        perm = np.concatenate([G_ * GROUP + np.random.default_rng(G_).permutation(GROUP) for G_ in np.random.default_rng(1).permutation(i // GROUP)]).astype(np.int32)
        for M in (1, 8, 8192):
            x = xt(M, i)
            y = torch.empty((M, o), dtype=torch.float16, device="cuda")
            n = 30 if M < 100 else 3

            def run_lin():
                for k in range(n):
                    hs3[k % 3].bpdq_linear(x.data_ptr(), y.data_ptr(), M, sp)
            run_lin()
            base = event_time_ms(torch, run_lin, stream) / n
            for h in hs3:
                h.bpdq_set_input_permutation(perm)
            run_lin()
            with_perm = event_time_ms(torch, run_lin, stream) / n
            for h in hs3:
                h.bpdq_set_input_permutation(None)
                h.bpdq_set_bias(np.zeros(o, dtype=np.uint16))
            run_lin()
            with_bias = event_time_ms(torch, run_lin, stream) / n
            for h in hs3:
                h.bpdq_set_bias(None)
            rec[f"M{M}"] = {"us_plain": base * 1e3, "us_with_permutation": with_perm * 1e3, "us_with_bias": with_bias * 1e3}
        out["gate_K2_permutation_and_bias_cost"] = rec
        up3 = [binding.Handle(o, i, K, GROUP, None, 1410 + c, 16) for c in range(3)]
        recs = {}
        for M in (1, 8):
            x = xt(M, i)
            hh = torch.empty((M, o), dtype=torch.float16, device="cuda")
            n = 30

            def run_unit():
                for k in range(n):
                    binding.bpdq_gate_up_swiglu(hs3[k % 3], up3[k % 3], x.data_ptr(), hh.data_ptr(), M, sp)
            run_unit()
            ms = event_time_ms(torch, run_unit, stream) / n
            b = 2 * useful_bytes(o, i, K, GROUP, M) - M * i * 2 - M * o * 2
            recs[f"M{M}"] = {"us": ms * 1e3, "gbs": b / (ms * 1e-3) / 1e9, "frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        out["gate_up_gated_unit_K2"] = recs
        for h in hs3 + up3:
            h.bpdq_destroy()
    # structured planes: a 7B-shaped gate projection quantized by the data-free producer (most significant bits of
    # Gaussian weights with outliers, fitted coefficients) against the same shape with random planes
    for K in (2,):
        o, i = 18944, 3584
        rng = np.random.default_rng(7)
        w = rng.normal(0, 0.02, size=(o, i)).astype(np.float32)
        w[rng.random(w.shape) < 0.002] *= 10.0
        bits, coef = binding.bpdq_quantize_datafree(w, K, GROUP)
        blob = binding.bpdq_pack(bits, coef, GROUP)
        del w, bits, coef
        copies = 8
        structured = [binding.Handle(o, i, K, GROUP, blob, 0, 8) for _ in range(copies)]
        random_ = [binding.Handle(o, i, K, GROUP, None, 1500 + c, 8) for c in range(copies)]
        rec = {"shape": [o, i], "K": K, "copies_rotated": copies}
        for M in (1, 8):
            x = xt(M, i)
            y = torch.empty((M, o), dtype=torch.float16, device="cuda")
            n = 80
            for tag, hl in (("structured", structured), ("random", random_)):
                def run_s():
                    for k in range(n):
                        hl[k % copies].bpdq_linear(x.data_ptr(), y.data_ptr(), M, sp)
                run_s()
                rec[f"us_{tag}_M{M}"] = event_time_ms(torch, run_s, stream) / n * 1e3
        out["structured_planes_7b_gate_K2"] = rec
        for h in structured + random_:
            h.bpdq_destroy()

    # a decoder layer with a few tokens in flight (M = 4, 8, 16): the grouping a decoder allows, one bpdq_linear_batch
    # call per group (the few-token kernel takes them above two tokens)
    for K in (2, 3):
        copies = 3
        layers = [[binding.Handle(o, i, K, GROUP, None, 1300 + 10 * c + li, 16) for li, (_, o, i) in enumerate(shapes)] for c in range(copies)]
        for M in (4, 8, 16):
            xs = {8192: xt(M, 8192), 29568: xt(M, 29568)}
            ys = [torch.empty((M, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes]
            b = layer_bytes(shapes, K, M)
            n = 30

            def run_few():
                for k in range(n):
                    hs_ = layers[k % copies]
                    for grp in ([0, 1, 2], [3], [4, 5], [6]):
                        binding.bpdq_linear_batch([hs_[j] for j in grp], [xs[hs_[j].in_].data_ptr() for j in grp],
                                                  [ys[j].data_ptr() for j in grp], M, sp)
            run_few()
            ms = event_time_ms(torch, run_few, stream) / n
            out[f"few_token_layer_decoder_groups_K{K}_M{M}"] = {"launches_per_layer": 4, "us_per_layer": ms * 1e3, "gbs": b / (ms * 1e-3) / 1e9,
                                                                "frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        for L in layers:
            for h in L:
                h.bpdq_destroy()
    return out


def full_stack_section(torch, binding, peaks, sp, stream, n_layers=80, group=GROUP):
    """All linears of an 80-layer 72B-shaped stack (K = 2: about 20.8 GB packed at g = 128, 19.2 GB at g = 256), one token
    through each."""
    shapes, K = synth.QWEN25_72B_LAYER, 2
    hs = []
    for layer in range(n_layers):
        for li, (_, o, i) in enumerate(shapes):
            hs.append(binding.Handle(o, i, K, group, None, synth.linear_seed(5, layer, li, K), 1))
    xs = {i: torch.from_numpy(synth.activations(9, 1, i).view(np.int16).copy()).cuda().view(torch.float16) for i in (8192, 29568)}
    ys = {o: torch.empty((1, o), dtype=torch.float16, device="cuda") for o in sorted({o for _, o, _ in shapes})}

    def sweep():
        for h in hs:
            h.bpdq_linear(xs[h.in_].data_ptr(), ys[h.out].data_ptr(), 1, sp)
    sweep()
    ms = sorted(event_time_ms(torch, sweep, stream) for _ in range(3))[1]
    b = n_layers * sum(useful_bytes(o, i, K, group, 1) for _, o, i in shapes)
    res = {"layers": n_layers, "group": group, "linears": len(hs), "packed_gb": sum(h.packed_bytes for h in hs) / 1e9, "ms_per_sweep": ms,
           "gbs": b / (ms * 1e-3) / 1e9, "frac_measured": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    # the same sweep as one bpdq_linear_batch call per layer (every linear of a batch needs an output of its own)
    n = len(shapes)
    ys_each = [torch.empty((1, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes]
    x_ptrs = [xs[i].data_ptr() for _, _, i in shapes]
    y_ptrs = [y.data_ptr() for y in ys_each]

    def sweep_batched():
        for layer in range(n_layers):
            binding.bpdq_linear_batch(hs[layer * n:(layer + 1) * n], x_ptrs, y_ptrs, 1, sp)
    sweep_batched()
    ms_b = sorted(event_time_ms(torch, sweep_batched, stream) for _ in range(3))[1]
    res["one_launch_per_layer"] = {"launches": n_layers, "ms_per_sweep": ms_b, "gbs": b / (ms_b * 1e-3) / 1e9,
                                   "frac_measured": b / (ms_b * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    # and in the grouping a decoder allows: {q, k, v} {o} {gate, up} {down}, four launches per layer
    groups = [[0, 1, 2], [3], [4, 5], [6]]

    def sweep_groups():
        for layer in range(n_layers):
            for grp in groups:
                binding.bpdq_linear_batch([hs[layer * n + j] for j in grp], [x_ptrs[j] for j in grp], [y_ptrs[j] for j in grp], 1, sp)
    sweep_groups()
    ms_g = sorted(event_time_ms(torch, sweep_groups, stream) for _ in range(3))[1]
    res["decoder_groups"] = {"launches": n_layers * len(groups), "ms_per_sweep": ms_g, "gbs": b / (ms_g * 1e-3) / 1e9,
                             "frac_measured": b / (ms_g * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    for h in hs:
        h.bpdq_destroy()
    return res


def run_case(a):
    """One kernel of the library a few times on one synthetic linear (or the 72B-shaped layer in one batched launch):
    the small, single-kernel command that profiler captures are taken from.  Prints the median launch time."""
    import torch
    from paper_2602_04163_b200 import binding
    kernels = {"auto": binding.KERNEL_AUTO, "gemv": binding.KERNEL_GEMV, "gemm": binding.KERNEL_GEMM,
               "simple": binding.KERNEL_GEMV_SIMPLE, "few": binding.KERNEL_FEW}
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if a.flush_l2 else None
    M = max(1, a.M)
    if a.case == "layer72b":
        shapes = synth.QWEN25_72B_LAYER
        hs = [binding.Handle(o, i, a.K, a.group, None, a.seed + li, M) for li, (_, o, i) in enumerate(shapes)]
        xs = {i: torch.from_numpy(synth.activations(a.seed + 9, M, i).view(np.int16).copy()).cuda().view(torch.float16)
              for i in sorted({i for _, _, i in shapes})}
        ys = [torch.empty((M, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes]

        def call():
            binding.bpdq_linear_batch(hs, [xs[h.in_].data_ptr() for h in hs], [y.data_ptr() for y in ys], M, sp)
        what = f"layer72b batch K={a.K} g={a.group} M={M}"
    else:
        hs = [binding.Handle(a.out, a.in_, a.K, a.group, None, a.seed, M)]
        x = torch.from_numpy(synth.activations(a.seed + 1, M, a.in_).view(np.int16).copy()).cuda().view(torch.float16)
        y = torch.empty((M, a.out), dtype=torch.float16, device="cuda")
        w = torch.empty((a.out, a.in_), dtype=torch.float16, device="cuda") if a.case == "dequant" else None

        def call():
            if a.case == "dequant":
                hs[0].bpdq_dequant(w.data_ptr(), sp)
            else:
                hs[0].bpdq_linear_ex(x.data_ptr(), y.data_ptr(), M, kernels[a.case], sp)
        what = f"{a.case} out={a.out} in={a.in_} K={a.K} g={a.group} M={M}"
    times = []
    for _ in range(a.iters):
        if flush is not None:
            flush.zero_()
        times.append(event_time_ms(torch, call, stream))
    hs[0].bpdq_get_status(sp)
    times.sort()
    med = times[len(times) // 2]
    packed = sum(h.packed_bytes for h in hs)
    print(f"{what}: median {med * 1e3:.1f} us over {a.iters} launches; packed {packed / 1e6:.1f} MB -> {packed / med / 1e6:.0f} GB/s")
    for h in hs:
        h.bpdq_destroy()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--case", default=None, choices=["auto", "gemv", "few", "gemm", "simple", "dequant", "layer72b"],
                    help="run one kernel on one linear instead of the benchmark (for profilers)")
    ap.add_argument("--out", type=int, default=29568)
    ap.add_argument("--in", dest="in_", type=int, default=8192)
    ap.add_argument("--K", type=int, default=2)
    ap.add_argument("--group", type=int, default=128)
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--flush-l2", action="store_true", help="with --case: write 256 MB between launches")
    args = ap.parse_args()
    if args.case:
        run_case(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.warmup < 3:
        args.warmup = 3
    run_cuda(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
