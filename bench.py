#!/usr/bin/env python
"""Benchmark of the BITCOS GEMV hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Workload (N = 1): one decode token (batch 1) through the seven ternary GEMVs of one
BitNet-b1.58-2B-shaped decoder layer -- q/o 2560x2560, k/v 640x2560, gate/up 6912x2560,
down 2560x6912 -- zero density 0.4219, group 128, bf16 group scales, int8 activations.
A "step" is that whole layer pass: seven bitcos_gemv launches.  Inputs are seeded synthetic
tensors; the packed layer is replicated so that consecutive steps never find their weights
in L2 (rotation set > 4x L2).

Prints one JSON line.  `value` is microseconds per token with everything resident in HBM;
`e2e` is the same through the host-buffer entry point with the host<->device copies of the
activations and outputs inside the timed region; `roofline` is the achieved algorithmic
bytes per second of the bitcos_gemv kernel against the measured HBM peak; `cpu_baseline` is
the CPU oracle timed on this machine's host cores.  With --gpus N every rank runs its own
replica of the workload (the path has no cross-GPU exchange).
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

import datagen  # noqa: E402

METRIC = "bitcos_gemv_us_per_token"
UNIT = "us"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
# roofline.traffic comes from the ncu summary of this command under profiles/: the file carries a line
#   dram_bytes_per_step = <dram__bytes_read.sum + dram__bytes_write.sum of the launches of one step>  commit = <hash>
TRAFFIC_PROFILE = os.path.join("profiles", "launch_list_and_dram_traffic_bitnet2b_layer_bench_default.md")


def ncu_traffic():
    """(bytes per step, source) of the default step's DRAM traffic as the committed ncu summary states it;
    (None, reason) if the summary is missing or carries no figure."""
    import re
    path = os.path.join(ROOT, TRAFFIC_PROFILE)
    try:
        with open(path) as f:
            text = f.read()
    except OSError:
        return None, f"{TRAFFIC_PROFILE} missing"
    m = re.search(r"dram_bytes_per_step\s*=\s*(\d+)\s+commit\s*=\s*([0-9a-f]{7,40})", text)
    if not m:
        return None, f"{TRAFFIC_PROFILE} carries no dram_bytes_per_step line"
    return int(m.group(1)), f"{TRAFFIC_PROFILE} (ncu capture at commit {m.group(2)})"


def layer_config():
    cfg = datagen.CONFIG_BITNET_2B
    return cfg, "bitnet-b1.58-2B decoder layer, 7 GEMVs, batch 1, z=0.4219, group 128"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def generate_layer(cfg, config_index=1):
    """Seeded trits, scales and activations for every matrix of the layer (host numpy)."""
    out = []
    for i, (name, M, K) in enumerate(cfg["shapes"]):
        seed = datagen.config_seed(config_index, i)
        W = datagen.trits(seed, M, K, cfg["z"])
        S = datagen.scales(seed, M, K)
        x, xs = datagen.activations(seed, 1, K)
        out.append({"name": name, "M": M, "K": K, "W": W, "S": S, "x": x, "xs": xs})
    return out


def algorithmic_bytes(M, K, nnz, batch, fmt="bitcos"):
    """Bytes one GEMV must move: packed weights + scales + offsets + activations + outputs."""
    Mp = (M + 31) // 32 * 32
    G = K // 128
    scales = 2 * Mp * G
    io = batch * (K + 4) + 4 * batch * M
    if fmt == "bitcos":
        return Mp * K // 8 + (nnz + 7) // 8 + scales + 4 * (Mp // 32 * G + 1) + io
    if fmt == "trit5":
        return Mp * ((26 * G + 3) // 4) * 4 + scales + io
    return Mp * K // 4 + scales + io


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------------
def oracle_layer_pass(layer, packed):
    import oracle
    for m, p in zip(layer, packed):
        oracle.gemv_packed(oracle.FORMAT_BITCOS, p.bitmap, p.signs, p.tile_off, m["S"], m["x"], m["xs"], m["M"], m["K"])


def oracle_pack_layer(layer):
    import oracle
    return [oracle.bitcos_pack(m["W"]) for m in layer]


def run_reference(args):
    """Times the oracle on the host cores.  Each step is a bounded sample of the layer pass: the
    first rows of every matrix (a multiple of 32), sized from one calibration pass so that the
    whole run stays within about two minutes; the reported time is scaled to the full layer."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, workload = layer_config()
    layer = generate_layer(cfg)
    packed = oracle_pack_layer(layer)
    cores = oracle.threads()
    t0 = time.perf_counter()
    oracle_layer_pass(layer, packed)
    full_pass = time.perf_counter() - t0
    frac = min(1.0, 120.0 / (full_pass * (args.steps + args.warmup)))
    sample = []
    for m in layer:
        rows = min(m["M"], max(32, int(m["M"] * frac) // 32 * 32))
        sample.append({**m, "M": rows, "W": m["W"][:rows], "S": m["S"][:rows]})
    frac = sum(s["M"] * s["K"] for s in sample) / sum(m["M"] * m["K"] for m in layer)
    spacked = oracle_pack_layer(sample)
    for _ in range(args.warmup):
        oracle_layer_pass(sample, spacked)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_layer_pass(sample, spacked)
    dt = time.perf_counter() - t0
    us = dt / args.steps * 1e6 / frac
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": workload, "batch": 1},
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"each step = the first {frac:.4f} of every matrix's rows (whole layer = 69.5 M "
                                   "weights), time scaled to the full layer: BITCOS decode bit by bit, dense int32 "
                                   "dot per group, double scale-and-sum"},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# Ranks: one process per GPU, independent replicas of the same workload (the path has no exchange
# step).  The only communication is the barrier around the timed region and the maximum over the
# ranks' times.
# ---------------------------------------------------------------------------------------------
class Ranks:
    """Process group plumbing of the benchmark: world size and rank from the launcher's environment,
    a barrier, and the maximum of a per-rank number.  backend "nccl" on GPUs; "gloo" lets the same
    code run on CPU (the tests do that with two processes)."""

    def __init__(self, backend="nccl", device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max(self, value):
        """Largest `value` over all ranks (every rank gets it)."""
        if self.dist is None:
            return float(value)
        import torch
        t = torch.tensor([float(value)], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None


def whole_job_value(us_per_step, world):
    """Time per token of the whole job: every replica finishes one token per step."""
    return us_per_step / world


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------
def run_cuda(args):
    import torch
    import paper_2609_16338_b200 as bc
    from paper_2609_16338_b200 import build as lib_build

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    ranks = Ranks("nccl", torch.device("cuda", local_rank))
    world, rank = ranks.world, ranks.rank
    if rank == 0:
        lib_build.build()
    ranks.barrier()
    bc.load_library()
    L = bc.load_library()

    cfg, workload = layer_config()
    layer = generate_layer(cfg)
    host_packed = [bc.bitcos_pack(m["W"], m["S"]) for m in layer]
    layer_bytes = sum(algorithmic_bytes(m["M"], m["K"], p.nnz, 1) for m, p in zip(layer, host_packed))
    packed_bytes = sum(p.payload_bytes() for p in host_packed)
    copies = max(2, int(np.ceil(4.2 * L2_BYTES / packed_bytes)))

    base = [p.to_device() for p in host_packed]
    replicas = [base] + [[w.clone() for w in base] for _ in range(copies - 1)]
    xs_dev = [(torch.from_numpy(m["x"]).cuda(), torch.from_numpy(m["xs"]).cuda()) for m in layer]
    ys = [torch.empty((1, m["M"]), dtype=torch.float32, device="cuda") for m in layer]
    wss = [bc.make_workspace(m["M"], m["K"]) for m in layer]

    sides = [torch.cuda.Stream(), torch.cuda.Stream()]
    # fused launches: GEMVs that read the same input and do not depend on one another share a launch
    groups = [[0, 1, 2], [3], [4, 5], [6]]
    multi = [[bc.MultiJobs([(rep[j], xs_dev[j][0], xs_dev[j][1], ys[j], wss[j]) for j in g]) for g in groups]
             for rep in replicas]

    # what each launch asks to be brought into L2: the matrices of the launch after it (the first
    # launch of the next layer -- the next rotated copy -- after the last)
    def later(c, gi, d):
        g = gi + d
        return [replicas[(c + g // len(groups)) % copies][j] for j in groups[g % len(groups)]]
    nexts = [[bc.NextWeights([w for d in args.prefetch_depth for w in later(c, gi, d)]) for gi in range(len(groups))]
             for c in range(copies)]
    # ... and what each launch is told runs directly before it (shapes only)
    prevs = [bc.NextWeights([base[j] for j in groups[gi - 1]]) for gi in range(len(groups))]

    phases = [p for p, g in enumerate(groups) for _ in g]
    order = [j for g in groups for j in g]
    phased = [bc.PhasedJobs([(rep[j], xs_dev[j][0], xs_dev[j][1], ys[j], wss[j]) for j in order], phases) for rep in replicas]

    def step(i):
        """One layer pass: q | k | v, then o, then gate | up, then down.  GEMVs that read the same
        input have no dependency on one another and are launched on forked streams (parallel
        branches of the CUDA graph); the rest follow in order."""
        rep = replicas[i % copies]

        def run(j):
            bc.bitcos_gemv(rep[j], xs_dev[j][0], xs_dev[j][1], y=ys[j], workspace=wss[j])

        if args.serial:
            for j in range(len(layer)):
                run(j)
            return
        if args.launch == "phased":
            bc.bitcos_gemv_phased(phased[i % copies])
            return
        if not args.branches:
            for gi, mj in enumerate(multi[i % copies]):
                bc.bitcos_gemv_multi(mj, next=nexts[i % copies][gi] if args.prefetch and gi in args.prefetch_launches else None,
                                     prev=prevs[gi] if args.chain_hint else None)
            return
        cur = torch.cuda.current_stream()
        for sd in sides:
            sd.wait_stream(cur)
        run(0)
        with torch.cuda.stream(sides[0]):
            run(1)
        with torch.cuda.stream(sides[1]):
            run(2)
        cur.wait_stream(sides[0])
        cur.wait_stream(sides[1])
        run(3)
        sides[0].wait_stream(cur)
        run(4)
        with torch.cuda.stream(sides[0]):
            run(5)
        cur.wait_stream(sides[0])
        run(6)

    # parity spot check of what is being timed (first replica, against the oracle, rank 0)
    step(0)
    torch.cuda.synchronize()
    if rank == 0:
        for m, y in zip(layer, ys):
            assert_matches_oracle(y, m["W"], m["S"], m["x"], m["xs"], f"layer pass, {m['name']}")

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()

    if args.profile_quant:
        # for profilers: plain stream launches of the layer pass from bf16 activations, nothing else
        step_q, step_b = quantised_layer_steps(bc, torch, layer, groups, replicas, ys, wss)
        run = step_q if args.profile_quant == "chain" else step_b
        for i in range(args.steps):
            run(i)
        torch.cuda.synchronize()
        status = max(bc.workspace_status(w) for w in wss)
        if rank == 0:
            print(json.dumps({"profile_quant": args.profile_quant, "steps": args.steps, "status": status}))
        ranks.close()
        return

    # Capture the rotation as CUDA graphs so that the host's launch cost is not what is timed.
    stream = torch.cuda.Stream()
    graphs = {}

    def capture(n_steps, first):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                for i in range(n_steps):
                    step(first + i)
        return g

    class Eager:
        """Stand-in for a captured graph: launches the steps directly on the current stream."""

        def __init__(self, n_steps):
            self.n = n_steps

        def replay(self):
            for i in range(self.n):
                step(i)

    # One graph holds exactly --steps layer passes (rotating over the weight copies).  It is replayed
    # back to back at least 30 times (and for at least a second, so that the clock sampler sees the
    # load); every replay is bracketed by CUDA events on the launching stream, and the reported time
    # is the median replay.  The clock sampler runs from before the untimed replays to the end.
    sampler = ClockSampler(local_rank)
    sampler.start()
    with torch.cuda.stream(stream):
        timed_graph = Eager(args.steps) if args.no_graph else capture(args.steps, 0)
        for _ in range(3):
            timed_graph.replay()
        stream.synchronize()
    ranks.barrier()
    torch.cuda.synchronize()
    replay_ms = []
    t_begin = time.time()
    with torch.cuda.stream(stream):
        while len(replay_ms) < 30 or (time.time() - t_begin < 1.0 and len(replay_ms) < 2000):
            evs = []
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                timed_graph.replay()
                e1.record(stream)
                evs.append((e0, e1))
            stream.synchronize()
            replay_ms += [a.elapsed_time(b) for a, b in evs]
    torch.cuda.synchronize()
    ranks.barrier()
    clocks = sampler.stop()
    ms = ranks.max(float(np.median(replay_ms)))
    ms_min, ms_max = ranks.max(float(np.min(replay_ms))), ranks.max(float(np.max(replay_ms)))

    # ---- end to end: host buffers through bitcos_gemv_host, copies inside the timed region ----
    stagings = [torch.empty(bc.bitcos_gemv_host_staging_bytes(m["M"], m["K"], 1), dtype=torch.uint8, device="cuda")
                for m in layer]
    xh = [torch.from_numpy(m["x"]).pin_memory() for m in layer]
    xsh = [torch.from_numpy(m["xs"]).pin_memory() for m in layer]
    yh = [torch.empty((1, m["M"]), dtype=torch.float32).pin_memory() for m in layer]
    xh_np, xsh_np, yh_np = [t.numpy() for t in xh], [t.numpy() for t in xsh], [t.numpy() for t in yh]

    host_multi = [[bc.MultiHostJobs([(rep[j], xh_np[j], xsh_np[j], yh_np[j], stagings[j], wss[j]) for j in g])
                   for g in groups] for rep in replicas]

    # one call per step: one pinned block in, the four launches, one pinned block out, one wait
    host_phases = [bc.HostPhases([(rep[j], wss[j]) for j in order], phases) for rep in replicas]
    for hp in host_phases:
        for n, j in enumerate(order):
            hp.x[n][:] = layer[j]["x"]
            hp.x_scale[n][:] = layer[j]["xs"]

    def e2e_step(i):
        if args.serial or args.branches:
            rep = replicas[i % copies]
            for j in range(len(layer)):
                bc.bitcos_gemv_host(rep[j], xh_np[j], xsh_np[j], yh_np[j], stagings[j], wss[j])
            return
        if args.e2e_per_phase:
            for mj in host_multi[i % copies]:
                bc.bitcos_gemv_multi_host(mj)
            return
        host_phases[i % copies].run()

    e2e_steps = 0 if args.no_e2e else min(args.steps, 200)
    e2e_us, e2e_chunks = float("nan"), []
    if e2e_steps:
        # (three visits per weight copy: the host entry point enqueues a step directly when it first sees its
        # arguments, records it the second time and replays the record from then on)
        for i in range(max(10, 3 * copies)):
            e2e_step(i)
        torch.cuda.synchronize()
        # wall clock around chunks of steps (every step ends with its own stream wait); the median chunk
        # is reported, so that a burst of other work on the host does not decide the figure
        for c in range(10):
            t0 = time.perf_counter()
            for i in range(e2e_steps):
                e2e_step(c * e2e_steps + i)
            e2e_chunks.append((time.perf_counter() - t0) / e2e_steps * 1e6)
        torch.cuda.synchronize()
        e2e_us = float(np.median(e2e_chunks))
    e2e_us = ranks.max(e2e_us)
    if args.serial or args.branches or args.e2e_per_phase:
        h2d = sum(m["K"] + 4 for m in layer)
        d2h = sum(4 * m["M"] for m in layer)
    else:
        h2d, d2h = host_phases[0].in_bytes, host_phases[0].out_bytes      # the two blocks as copied (16-byte padding included)

    if rank != 0:
        ranks.close()
        return

    # ---- every launch of a step on its own: idle GPU, cold L2, events around the one launch ----
    isolated_us = None
    phased_us = None
    if not args.no_detail:
        flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
        isolated_us = []
        for gi in range(len(groups)):
            ts = []
            for r in range(12):
                flush_buf.zero_()
                torch.cuda.synchronize()
                with torch.cuda.stream(stream):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    bc.bitcos_gemv_multi(multi[r % copies][gi])
                    b.record(stream)
                    stream.synchronize()
                ts.append(a.elapsed_time(b) * 1e3)
            isolated_us.append(float(np.median(ts)))
        # the whole layer pass as ONE launch with the dependencies enforced inside it
        phased_us = graph_time_us(torch, stream, lambda i: bc.bitcos_gemv_phased(phased[i]), copies, launches=copies)

    # ---- the same seven products as ONE launch per step (what the launch structure costs) ----
    one_launch_us = None
    if not args.no_detail:
        all_jobs = [bc.MultiJobs([(rep[j], xs_dev[j][0], xs_dev[j][1], ys[j], wss[j]) for j in range(len(layer))])
                    for rep in replicas]
        one_launch_us = graph_time_us(torch, stream, lambda i: bc.bitcos_gemv_multi(all_jobs[i]), copies, launches=copies)

    # ---- the layer pass with an activation quantiser in front of each of its four launches ----
    # (bf16 activations -> int8 and one scale per token, then the fused launch that reads them)
    with_quant_us = fused_quant_us = None
    if not args.no_detail and not (args.serial or args.branches):
        step_q, step_b = quantised_layer_steps(bc, torch, layer, groups, replicas, ys, wss)
        with_quant_us = graph_time_us(torch, stream, step_q, copies, launches=copies)
        fused_quant_us = graph_time_us(torch, stream, step_b, copies, launches=copies)

    # ---- per-shape detail: each format on each shape, rotated copies, CUDA graph of 64 launches ----
    detail = shape_detail(bc, torch, layer, host_packed, stream) if not args.no_detail else None

    # ---- CPU baseline: the oracle on the host cores, bounded sample ----
    import oracle
    reps, cpu_us, cpu1_us = 0, float("nan"), float("nan")
    if not args.no_cpu_baseline:
        o_packed = oracle_pack_layer(layer)
        t0 = time.perf_counter()
        while True:
            oracle_layer_pass(layer, o_packed)
            reps += 1
            if time.perf_counter() - t0 > 10.0 or reps >= 20:
                break
        cpu_us = (time.perf_counter() - t0) / reps * 1e6
        # the same on one thread (two passes)
        all_threads = oracle.threads()
        oracle.set_threads(1)
        t0 = time.perf_counter()
        for _ in range(2):
            oracle_layer_pass(layer, o_packed)
        cpu1_us = (time.perf_counter() - t0) / 2 * 1e6
        oracle.set_threads(all_threads)

    peak, which = measured_peaks()
    us_per_step = ms * 1e3 / args.steps
    launches_per_step = 7 if (args.serial or args.branches) else 1 if args.launch == "phased" else len(groups)
    traffic_step, traffic_src = ncu_traffic()
    n_launch = launches_per_step * args.steps
    achieved = layer_bytes * args.steps / (ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": whole_job_value(us_per_step, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": us_per_step / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": workload, "batch": 1, "weights": int(sum(m["M"] * m["K"] for m in layer)),
                   "packed_bytes_per_step": int(packed_bytes), "algorithmic_bytes_per_step": int(layer_bytes),
                   "l2_policy": f"{copies} rotated copies of the packed layer ({copies * packed_bytes / 2**20:.0f} MiB)"
                                " so no step finds its weights in L2",
                   "launch": (("plain stream launches; " if args.no_graph else "CUDA graphs of the rotation; ")
                              + ("7 launches per step, in sequence" if args.serial else
                                 "7 launches per step: q|k|v on parallel branches, o, gate|up on parallel branches, down"
                                 if args.branches else
                                 "4 launches per step through bitcos_gemv_multi: q+k+v, o, gate+up, down (GEMVs that "
                                 "read the same input share a launch)"
                                 + ("; launches " + ",".join(str(g + 1) for g in args.prefetch_launches)
                                    + " of the step also ask for the NEXT launch's packed weights to be brought into L2"
                                      " (bitcos_gemv_multi_chained): every byte still comes from device memory"
                                      " once per step" if args.prefetch and args.launch == "multi" else "")
                                 + ("; every launch is told which launch runs directly before it (blocks that start late take"
                                    " fewer work items; results unchanged)" if args.chain_hint and args.launch == "multi" else ""))
                              + "; programmatic dependent launch between consecutive kernels of a stream"),
                   "replicas": world},
        "achieved_gbs": achieved,
        "frac_of_8tbs": achieved / 8000.0,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (traffic_step / launches_per_step) if (traffic_step and launches_per_step == 4 and args.launch == "multi") else None,
                     "traffic_source": traffic_src, "peak_source": f"{which} (STREAM-style copy)",
                     "kernel": "gemv_kernel<bitcos, 1 token>" if launches_per_step == 7 else "gemv_phased_kernel<1 token>" if launches_per_step == 1 else "gemv_multi_kernel<1 token>",
                     "launches": n_launch,
                     "avg_launch_us": ms * 1e3 / n_launch,
                     "algorithmic_bytes_per_launch": layer_bytes / launches_per_step},
        "cpu_baseline": {"value": cpu_us, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "one_thread_us": cpu1_us,
                         "sample": f"{reps} full layer passes (7 GEMVs, 69.5 M weights each): BITCOS decode bit by "
                                   "bit, dense int32 dot per group, double scale-and-sum"},
        "e2e": {"value": whole_job_value(e2e_us, world), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "chunks": len(e2e_chunks), "statistic": "median chunk",
                "us_min": min(e2e_chunks) if e2e_chunks else None, "us_max": max(e2e_chunks) if e2e_chunks else None,
                "path": ("bitcos_gemv_host per GEMV: pinned x -> device, kernel, y -> pinned host, stream wait"
                         if (args.serial or args.branches) else
                         "bitcos_gemv_multi_host, four calls per step, each: pinned x -> device, launch, y -> pinned host, stream wait"
                         if args.e2e_per_phase else
                         "bitcos_gemv_phases_host, one call per step: one pinned block with all activations -> device, "
                         "four launches (q+k+v, o, gate+up, down), all outputs -> one pinned block, one stream wait; "
                         "the library replays a step it has seen before as a recorded CUDA graph")},
        "gpu_launches": n_launch,
        "timing": {"replays": len(replay_ms), "steps_per_replay": args.steps, "statistic": "median replay",
                   "us_per_step_min": ms_min * 1e3 / args.steps, "us_per_step_max": ms_max * 1e3 / args.steps},
        "clocks": clocks,
    }
    line["two_term_roofline"] = two_term_roofline(bc, cfg["z"], peak, clocks.get("sm_mhz") or 1965.0)
    if detail is not None:
        line["isolated_launch_us"] = {"q+k+v": isolated_us[0], "o": isolated_us[1], "gate+up": isolated_us[2], "down": isolated_us[3],
                                      "note": "one launch on an idle GPU with L2 flushed, CUDA events directly around it "
                                              "(launch latency included, nothing overlaps)"}
        line["phased_launch_per_step"] = {
            "us": phased_us,
            "note": "bitcos_gemv_phased: the layer pass as one launch, phases q|k|v, o, gate|up, down, the dependency "
                    "between phases enforced by a device-side counter"}
        line["one_launch_per_step"] = {
            "us": one_launch_us, "gbs": layer_bytes / one_launch_us / 1e3, "frac": layer_bytes / one_launch_us / 1e3 / peak,
            "note": "all seven products of the layer in a single bitcos_gemv_multi launch: possible for independent "
                    "products only (in a decoder layer o follows attention over q, k, v and down follows gate and up), so "
                    "this is not the headline; it shows how much of the step is launch structure"}
        if with_quant_us is not None:
            line["layer_with_quantisers"] = {
                "us": with_quant_us,
                "note": "the timed step with bitcos_quantize_activations (bf16 -> int8, one scale per token) in front "
                        "of each of its four launches: eight kernels per step, each overlapping its start-up with the "
                        "kernel before it",
                "fused_us": fused_quant_us,
                "fused_note": "bitcos_gemv_multi_bf16: the same four launches as the timed step, reading bf16 activations "
                              "and quantising them per group of 128 inside the decoder warps"}
        line["shapes"] = detail
        line["batch"] = batch_detail(bc, torch, stream)
        line["activation_quant"] = quant_detail(bc, torch, stream)
    if detail is not None and not args.layer_only:
        # the other configurations: zero-density sweep, the Qwen3-32B-shaped layer at 1 to 16 tokens,
        # the grouped mixture-of-experts product
        line["density_sweep"] = sweep_detail(bc, torch, stream)
        line["qwen32b_layer"] = qwen32b_layer_detail(bc, torch, stream)
        line["moe"] = moe_detail(bc, torch, stream)
    if args.all_configs:
        line["device_pack"] = pack_detail(bc, torch)
    print(json.dumps(line))
    ranks.close()


def quantised_layer_steps(bc, torch, layer, groups, replicas, ys, wss):
    """The layer pass from bf16 activations, two ways.  step_q: bitcos_quantize_activations (one scale
    per token) in front of each fused launch, eight kernels per step.  step_b: the quantiser inside
    the products (bitcos_gemv_multi_bf16, scales per group of 128), four launches per step."""
    import datagen
    xb, qx, qs = [], [], []
    for gi, g in enumerate(groups):
        K = layer[g[0]]["K"]
        bits = datagen.activations_bf16(datagen.config_seed(1, 60 + gi), 1, K)
        xb.append(torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16))
        qx.append(torch.empty((1, K), dtype=torch.int8, device="cuda"))
        qs.append(torch.empty((1,), dtype=torch.float32, device="cuda"))
    multi_q = [[bc.MultiJobs([(rep[j], qx[gi], qs[gi], ys[j], wss[j]) for j in g]) for gi, g in enumerate(groups)]
               for rep in replicas]
    multi_b = [[bc.MultiJobs([(rep[j], xb[gi], None, ys[j], wss[j]) for j in g]) for gi, g in enumerate(groups)]
               for rep in replicas]

    def step_q(i):
        for gi, mj in enumerate(multi_q[i % len(multi_q)]):
            bc.bitcos_quantize_activations(xb[gi], 0, xq=qx[gi], x_scale=qs[gi])
            bc.bitcos_gemv_multi(mj)

    def step_b(i):
        for mj in multi_b[i % len(multi_b)]:
            bc.bitcos_gemv_multi_bf16(mj)

    return step_q, step_b


def two_term_roofline(bc, z, peak_gbs, sm_mhz, sms=148):
    """The paper's model T = max(B / beta, gamma) per 32 weights (Section III-B.1), evaluated on this
    GPU: gamma = measured cycles per 32 weights per multiprocessor with every operand on chip
    (bitcos_decode_probe, 20 decoder warps), beta = measured HBM bytes per clock per multiprocessor,
    B = bytes per 32 weights including the 16-bit group scale (and tile offsets for BITCOS)."""
    beta = peak_gbs * 1e9 / sms / (sm_mhz * 1e6)
    out = {"beta_bytes_per_clk_per_sm": beta, "sm_mhz": sm_mhz}
    for fmt, name, B in ((0, "bitcos", 4 + 4 * (1 - z) + 0.5 + 32 / 1024.0), (1, "trit5", 26 / 4.0 + 0.5), (2, "bit2", 8.5)):
        gamma = bc.bitcos_decode_probe(fmt, 20, 200, sms)
        mem = B / beta
        out[name] = {"bytes_per_32_weights": B, "memory_term_cycles": mem, "gamma_cycles": gamma,
                     "bound_by": "instructions" if gamma > mem else "memory",
                     "ceiling_gbs": B / max(mem, gamma) * sms * sm_mhz * 1e6 / 1e9}
    return out


def shape_detail(bc, torch, layer, host_packed, stream, launches=64):
    """Per distinct shape: microseconds and GB/s of bitcos / trit5 / bit2 on identical weights."""
    peak, _ = measured_peaks()
    seen, out = set(), []
    for m, p in zip(layer, host_packed):
        key = (m["M"], m["K"])
        if key in seen:
            continue
        seen.add(key)
        M, K = key
        st = bc.scales_tile(m["S"], M, K)
        fmts = {"bitcos": (p.to_device(), bc.bitcos_gemv), "trit5": (bc.plain_to_device(bc.trit5_pack(m["W"]), st, M, K), bc.trit5_gemv),
                "bit2": (bc.plain_to_device(bc.bit2_pack(m["W"]), st, M, K), bc.bit2_gemv)}
        x, xs = torch.from_numpy(m["x"]).cuda(), torch.from_numpy(m["xs"]).cuda()
        y = torch.empty((1, M), dtype=torch.float32, device="cuda")
        ws = bc.make_workspace(M, K)
        row = {"name": m["name"], "M": M, "K": K}
        for name, (Wd, f) in fmts.items():
            nbytes = algorithmic_bytes(M, K, p.nnz, 1, name)
            n_copies = max(2, int(np.ceil(4.2 * L2_BYTES / Wd.payload_bytes())))
            reps = [Wd] + [Wd.clone() for _ in range(n_copies - 1)]
            f(reps[0], x, xs, y=y, workspace=ws)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(stream):
                with torch.cuda.graph(g, stream=stream):
                    for i in range(launches):
                        f(reps[i % n_copies], x, xs, y=y, workspace=ws)
                g.replay()
                stream.synchronize()
                times = []
                for _ in range(5):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    g.replay()
                    e1.record(stream)
                    stream.synchronize()
                    times.append(e0.elapsed_time(e1) * 1e3 / launches)
            us = float(np.median(times))
            row[name] = {"us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak, "bytes": int(nbytes)}
            del reps, g
        row["speedup_vs_trit5"] = row["trit5"]["us"] / row["bitcos"]["us"]
        row["byte_ratio_trit5"] = row["trit5"]["bytes"] / row["bitcos"]["bytes"]
        row["speedup_vs_bit2"] = row["bit2"]["us"] / row["bitcos"]["us"]
        row["byte_ratio_bit2"] = row["bit2"]["bytes"] / row["bitcos"]["bytes"]
        out.append(row)
        torch.cuda.empty_cache()
    return out


def graph_time_us(torch, stream, launch, n_copies, launches=48, repeats=5):
    """Median microseconds per launch of `launch(i)` (i = which rotated copy), from CUDA graphs of
    `launches` launches replayed `repeats` times, events on the launching stream."""
    launch(0)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            for i in range(launches):
                launch(i % n_copies)
        g.replay()
        stream.synchronize()
        times = []
        for _ in range(repeats):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
            times.append(e0.elapsed_time(e1) * 1e3 / launches)
    return float(np.median(times))


def graph_time_flushed_us(torch, stream, launch, n_variants, flush, launches=24, repeats=5):
    """Like graph_time_us for launches whose working set is smaller than L2: every launch is
    preceded by a write of `flush` (larger than L2); the time of a graph holding only the flushes
    is subtracted."""
    launch(0)
    torch.cuda.synchronize()

    def timed(with_launch):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                for i in range(launches):
                    flush.zero_()
                    if with_launch:
                        launch(i % n_variants)
            g.replay()
            stream.synchronize()
            times = []
            for _ in range(repeats):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                g.replay()
                e1.record(stream)
                stream.synchronize()
                times.append(e0.elapsed_time(e1) * 1e3 / launches)
        return float(np.median(times))

    return timed(True) - timed(False)


def batch_detail(bc, torch, stream, M=8192, K=5120, z=0.4711):
    """Small-batch decode on one Qwen3-32B-shaped matrix (the q projection): the three formats at
    1, 2, 4, 8, 16 tokens; the weights are read once per call whatever the batch."""
    import datagen
    peak, _ = measured_peaks()
    seed = datagen.config_seed(3, 0)
    W, S = datagen.trits(seed, M, K, z), datagen.scales(seed, M, K)
    st = bc.scales_tile(S, M, K)
    packed = bc.bitcos_pack(W, S)
    fmts = {"bitcos": (packed.to_device(), bc.bitcos_gemv),
            "trit5": (bc.plain_to_device(bc.trit5_pack(W), st, M, K), bc.trit5_gemv),
            "bit2": (bc.plain_to_device(bc.bit2_pack(W), st, M, K), bc.bit2_gemv)}
    ws = bc.make_workspace(M, K)
    out = {"M": M, "K": K, "z": z, "rows": []}
    for B in (1, 2, 4, 8, 16):
        x, xs = datagen.activations(seed, B, K)
        xd, xsd = torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda()
        y = torch.empty((B, M), dtype=torch.float32, device="cuda")
        row = {"batch": B, "contraction": "dp4a" if B < 4 else "mma.m16n8k32.s8"}
        for name, (Wd, f) in fmts.items():
            n_copies = max(2, int(np.ceil(4.2 * L2_BYTES / Wd.payload_bytes())))
            reps = [Wd] + [Wd.clone() for _ in range(n_copies - 1)]
            us = graph_time_us(torch, stream, lambda i: f(reps[i], xd, xsd, y=y, workspace=ws), n_copies)
            nbytes = algorithmic_bytes(M, K, packed.nnz, B, name)
            row[name] = {"us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak,
                         "us_per_token": us / B}
            del reps
        out["rows"].append(row)
        torch.cuda.empty_cache()
    return out


def quant_detail(bc, torch, stream):
    """The quantised-activation front end: bf16 activations -> int8 quantiser (one scale per group
    of 128, or per token) -> product, on two matrices at 1, 4 and 16 tokens.  `chain` is one
    quantiser launch plus one product launch back to back on the stream (the product's start-up
    overlaps the quantiser); `gemv` is the product alone on ready int8 activations."""
    import datagen
    out = []
    for (M, K, z, ci) in ((2560, 6912, 0.4219, 1), (8192, 5120, 0.4711, 3)):
        seed = datagen.config_seed(ci, 40)
        W, S = datagen.trits(seed, M, K, z), datagen.scales(seed, M, K)
        packed = bc.bitcos_pack(W, S)
        Wd = packed.to_device()
        n_copies = max(2, int(np.ceil(4.2 * L2_BYTES / Wd.payload_bytes())))
        reps = [Wd] + [Wd.clone() for _ in range(n_copies - 1)]
        ws = bc.make_workspace(M, K)
        G = K // 128
        for B in (1, 2, 4, 8, 16):
            xb = torch.from_numpy(datagen.activations_bf16(seed + B, B, K).view(np.int16)).cuda().view(torch.bfloat16)
            q = torch.empty((B, K), dtype=torch.int8, device="cuda")
            sg = torch.empty((B, G), dtype=torch.float32, device="cuda")
            st = torch.empty((B,), dtype=torch.float32, device="cuda")
            y = torch.empty((B, M), dtype=torch.float32, device="cuda")
            bc.bitcos_quantize_activations(xb, 128, xq=q, x_scale=sg)
            bc.bitcos_quantize_activations(xb, 0, xq=q, x_scale=st)
            row = {"M": M, "K": K, "batch": B}
            row["gemv_us"] = graph_time_us(torch, stream, lambda i: bc.bitcos_gemv(reps[i], q, st, y=y, workspace=ws), n_copies)
            row["gemv_group_scales_us"] = graph_time_us(
                torch, stream, lambda i: bc.bitcos_gemv_group_scales(reps[i], q, sg, y=y, workspace=ws), n_copies)
            row["quantise_groups_us"] = graph_time_us(
                torch, stream, lambda i: bc.bitcos_quantize_activations(xb, 128, xq=q, x_scale=sg), 1)
            row["quantise_tokens_us"] = graph_time_us(
                torch, stream, lambda i: bc.bitcos_quantize_activations(xb, 0, xq=q, x_scale=st), 1)

            def chain_groups(i):
                bc.bitcos_quantize_activations(xb, 128, xq=q, x_scale=sg)
                bc.bitcos_gemv_group_scales(reps[i], q, sg, y=y, workspace=ws)

            def chain_tokens(i):
                bc.bitcos_quantize_activations(xb, 0, xq=q, x_scale=st)
                bc.bitcos_gemv(reps[i], q, st, y=y, workspace=ws)

            if B <= 2:
                # the quantiser inside the product's thread blocks (one and two tokens)
                row["gemv_bf16_us"] = graph_time_us(
                    torch, stream, lambda i: bc.bitcos_gemv_bf16(reps[i], xb, y=y, workspace=ws), n_copies)
            if B <= 8:
                # the 16-bit variant: weights rebuilt as +-s against the unquantised activations (tensor cores)
                row["gemv_blend_bf16_us"] = graph_time_us(
                    torch, stream, lambda i: bc.bitcos_gemv_blend_bf16(reps[i], xb, y=y, workspace=ws), n_copies)
            row["chain_groups_us"] = graph_time_us(torch, stream, chain_groups, n_copies)
            row["chain_tokens_us"] = graph_time_us(torch, stream, chain_tokens, n_copies)
            row["quantiser_bytes"] = int(B * K * 3 + 4 * B * G)
            out.append(row)
        del reps
        torch.cuda.empty_cache()
    return out


def pack_detail(bc, torch):
    """Device-side packing (set-up path): int8 trits + bf16 scales in device memory -> the BITCOS
    buffers.  Wall time of the whole call (three kernels, two stream waits, the sign vector cut to size), against
    the bytes it has to move once: the trits in, the packed buffers out."""
    import time
    import datagen
    peak, _ = measured_peaks()
    out = []
    for (M, K, z, ci) in ((8192, 5120, 0.4711, 3), (25600, 5120, 0.4711, 3)):
        seed = datagen.config_seed(ci, 50)
        W, S = datagen.trits(seed, M, K, z), datagen.scales(seed, M, K)
        Wt, St = torch.from_numpy(W).cuda(), torch.from_numpy(S.view(np.int16)).cuda()
        Wd = bc.bitcos_pack_device(Wt, St)
        torch.cuda.synchronize()
        times = []
        for _ in range(5):
            t0 = time.perf_counter()
            Wd = bc.bitcos_pack_device(Wt, St)
            times.append((time.perf_counter() - t0) * 1e6)
        us = float(np.median(times))
        nbytes = M * K + S.nbytes + Wd.payload_bytes()
        out.append({"M": M, "K": K, "us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak,
                    "bytes_once": int(nbytes), "note": "the trits are read twice (bitmap and counts, signs)"})
        del Wt, St, Wd
        torch.cuda.empty_cache()
    return out


def assert_matches_oracle(y, W, S, x, xs, what):
    """Every table times outputs that were compared with the oracle first (fp32 within 1e-5 of sum|terms|)."""
    import oracle
    _, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= 1e-5 * mag).all(), f"bench: {what} disagrees with the oracle"


def sweep_detail(bc, torch, stream):
    """Zero-density sweep (two matrix shapes, five densities, one token): the three formats on
    identical weights, realised gain against the byte ratio."""
    import datagen
    peak, _ = measured_peaks()
    out = []
    for si, (M, K) in enumerate(((4096, 12288), (12288, 4096))):
        ws = bc.make_workspace(M, K)
        for zi, z in enumerate((0.30, 0.375, 0.42, 0.47, 0.515)):
            seed = datagen.config_seed(2, 10 * si + zi)
            W, S = datagen.trits(seed, M, K, z), datagen.scales(seed, M, K)
            x, xs = datagen.activations(seed, 1, K)
            xd, xsd = torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda()
            y = torch.empty((1, M), dtype=torch.float32, device="cuda")
            st = bc.scales_tile(S, M, K)
            packed = bc.bitcos_pack(W, S)
            fmts = {"bitcos": (packed.to_device(), bc.bitcos_gemv),
                    "trit5": (bc.plain_to_device(bc.trit5_pack(W), st, M, K), bc.trit5_gemv),
                    "bit2": (bc.plain_to_device(bc.bit2_pack(W), st, M, K), bc.bit2_gemv)}
            row = {"M": M, "K": K, "z": z, "z_realised": 1.0 - packed.nnz / float(M * K)}
            for name, (Wd, f) in fmts.items():
                n_copies = max(2, int(np.ceil(4.2 * L2_BYTES / Wd.payload_bytes())))
                reps = [Wd] + [Wd.clone() for _ in range(n_copies - 1)]
                f(reps[-1], xd, xsd, y=y, workspace=ws)
                torch.cuda.synchronize()
                assert_matches_oracle(y, W, S, x, xs, f"density sweep {M}x{K} z={z} {name}")
                us = graph_time_us(torch, stream, lambda i: f(reps[i], xd, xsd, y=y, workspace=ws), n_copies)
                nbytes = algorithmic_bytes(M, K, packed.nnz, 1, name)
                row[name] = {"us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak, "bytes": int(nbytes)}
                del reps
            row["speedup_vs_trit5"] = row["trit5"]["us"] / row["bitcos"]["us"]
            row["byte_ratio_trit5"] = row["trit5"]["bytes"] / row["bitcos"]["bytes"]
            row["speedup_vs_bit2"] = row["bit2"]["us"] / row["bitcos"]["us"]
            row["byte_ratio_bit2"] = row["bit2"]["bytes"] / row["bitcos"]["bytes"]
            out.append(row)
            torch.cuda.empty_cache()
    return out


def qwen32b_layer_detail(bc, torch, stream, z=0.4711):
    """One decode step through the seven linear maps of a Qwen3-32B-shaped layer at 1 to 16 tokens:
    four launches per step as in the headline (q+k+v, o, gate+up, down), two rotated copies of the
    101 MB layer (each launch's weights were last read two steps and more than L2's size ago)."""
    import datagen
    peak, _ = measured_peaks()
    shapes = [("q", 8192, 5120), ("k", 1024, 5120), ("v", 1024, 5120), ("o", 5120, 8192), ("gate", 25600, 5120),
              ("up", 25600, 5120), ("down", 5120, 25600)]
    host, dense = [], []
    for i, (_, M, K) in enumerate(shapes):
        seed = datagen.config_seed(3, i)
        dense.append((datagen.trits(seed, M, K, z), datagen.scales(seed, M, K)))
        host.append(bc.bitcos_pack(*dense[-1]))
    base = [h.to_device() for h in host]
    replicas = [base, [w.clone() for w in base]]
    wss = [bc.make_workspace(M, K) for (_, M, K) in shapes]
    groups = [[0, 1, 2], [3], [4, 5], [6]]
    out = []
    for B in (1, 2, 4, 8, 16):
        xs_dev, xs_host = [], []
        for i, (_, M, K) in enumerate(shapes):
            x, xs = datagen.activations(datagen.config_seed(3, i), B, K)
            xs_host.append((x, xs))
            xs_dev.append((torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda()))
        ys = [torch.empty((B, M), dtype=torch.float32, device="cuda") for (_, M, K) in shapes]
        multi = [[bc.MultiJobs([(rep[j], xs_dev[j][0], xs_dev[j][1], ys[j], wss[j]) for j in g]) for g in groups]
                 for rep in replicas]

        # every launch is told which launch runs before it and which matrices the next one reads (as in the headline)
        prevs = [bc.NextWeights([base[j] for j in groups[gi - 1]]) for gi in range(len(groups))]
        nexts = [[bc.NextWeights([replicas[(c + (gi + 1) // len(groups)) % len(replicas)][j] for j in groups[(gi + 1) % len(groups)]])
                  for gi in range(len(groups))] for c in range(len(replicas))]

        def step(i, hints=True):
            for gi, mj in enumerate(multi[i]):
                bc.bitcos_gemv_multi(mj, prev=prevs[gi] if hints else None, next=nexts[i][gi] if hints else None)

        step(1)
        torch.cuda.synchronize()
        for i, (nm, M, K) in enumerate(shapes):
            assert_matches_oracle(ys[i], dense[i][0], dense[i][1], xs_host[i][0], xs_host[i][1], f"qwen layer {nm} B={B}")
        us = graph_time_us(torch, stream, step, len(replicas), launches=8)
        us_plain = graph_time_us(torch, stream, lambda i: step(i, False), len(replicas), launches=8)
        nbytes = sum(algorithmic_bytes(M, K, h.nnz, B) for (_, M, K), h in zip(shapes, host))
        out.append({"batch": B, "us_per_step": us, "us_per_token": us / B, "gbs": nbytes / us / 1e3,
                    "frac": nbytes / us / 1e3 / peak, "bytes": int(nbytes), "us_per_step_without_hints": us_plain})
    return out


def run_profile_batch(args):
    """A few plain stream launches of one format at one batch size on the batch table's matrix
    (for profilers: no graphs, nothing else on the device).  Prints a small JSON line."""
    import torch
    import datagen
    import paper_2609_16338_b200 as bc
    from paper_2609_16338_b200 import build as lib_build
    lib_build.build()
    bc.load_library()
    M, K = (int(v) for v in args.profile_shape.split("x"))
    z, B = 0.4711, args.profile_batch
    seed = datagen.config_seed(3, 0)
    W, S = datagen.trits(seed, M, K, z), datagen.scales(seed, M, K)
    packed = bc.bitcos_pack(W, S)
    Wd = packed.to_device()
    n_copies = max(2, int(np.ceil(1.5 * L2_BYTES / Wd.payload_bytes())))
    reps = [Wd] + [Wd.clone() for _ in range(n_copies - 1)]
    x, xs = datagen.activations(seed, B, K)
    xd, xsd = torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda()
    y = torch.empty((B, M), dtype=torch.float32, device="cuda")
    ws = bc.make_workspace(M, K)
    if args.profile_entry == "blend":
        # the 16-bit variant: weights +-s against unquantised bf16 activations
        xb = torch.from_numpy(datagen.activations_bf16(seed, B, K).view(np.int16)).cuda().view(torch.bfloat16)

        def call(i):
            bc.bitcos_gemv_blend_bf16(reps[i % n_copies], xb, y=y, workspace=ws)
    else:
        def call(i):
            bc.bitcos_gemv(reps[i % n_copies], xd, xsd, y=y, workspace=ws)
    for i in range(3):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        call(i)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.steps
    print(json.dumps({"profile_batch": B, "entry": args.profile_entry, "M": M, "K": K, "launches": args.steps + 3, "us_per_launch_with_host_gaps": us,
                      "status": bc.workspace_status(ws)}))


def moe_detail(bc, torch, stream, E=128, top_k=8, z=0.3288):
    """Grouped product over the selected experts of a Qwen3-30B-A3B-shaped layer, the three formats on
    identical weights: gate/up (768 x 2048, the token's activations) and down (2048 x 768, one activation
    row per pair), 1 to 16 tokens, expert ids drawn without replacement per token.  The experts of one
    projection (46 MB packed) would fit in L2, so L2 is flushed before every launch and the routing is
    redrawn.  Every format's first draw is compared with the oracle before it is timed."""
    import datagen
    import oracle
    peak, _ = measured_peaks()

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a.view(np.int32) if a.dtype == np.uint32 else a)).cuda()

    out = []
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
    for name, (M, K) in (("gate/up", (768, 2048)), ("down", (2048, 768))):
        Ws = [datagen.trits(datagen.config_seed(4, e), M, K, z) for e in range(E)]
        Ss = [datagen.scales(datagen.config_seed(4, e), M, K) for e in range(E)]
        host = [bc.bitcos_pack(Ws[e], Ss[e]) for e in range(E)]
        sts = [bc.scales_tile(Ss[e], M, K) for e in range(E)]
        formats = (("bitcos", bc.DeviceExperts([h.to_device() for h in host]), bc.bitcos_gemv_grouped),
                   ("trit5", bc.DeviceExperts([bc.plain_to_device(bc.trit5_pack(Ws[e]), sts[e], M, K) for e in range(E)]), bc.trit5_gemv_grouped),
                   ("bit2", bc.DeviceExperts([bc.plain_to_device(bc.bit2_pack(Ws[e]), sts[e], M, K) for e in range(E)]), bc.bit2_gemv_grouped))
        for tokens in (1, 2, 4, 8, 16):
            draws = []
            for d in range(12):
                ids = datagen.expert_choices(1000 * tokens + d, tokens, E, top_k)
                pair_expert = ids.reshape(-1)
                if name == "gate/up":
                    pair_xrow = np.repeat(np.arange(tokens, dtype=np.int32), top_k)
                    x, xs = datagen.activations(17, tokens, K)
                else:
                    pair_xrow = np.arange(tokens * top_k, dtype=np.int32)
                    x, xs = datagen.activations(17, tokens * top_k, K)
                order, ge, gb, xr, mx = bc.group_pairs(pair_expert, pair_xrow)
                nb = {f: sum(algorithmic_bytes(M, K, host[e].nnz, int(gb[i + 1] - gb[i]), f) for i, e in enumerate(ge))
                      for f in ("bitcos", "trit5", "bit2")}
                draws.append((dev(ge), dev(gb), dev(xr), mx, len(ge), nb, (pair_expert[order], pair_xrow[order])))
            xd, xsd = dev(x), dev(xs)
            ws = bc.make_workspace(M, K, copies=max(d[4] for d in draws))
            y = torch.empty((tokens * top_k, M), dtype=torch.float32, device="cuda")
            _, y_ref, mag = oracle.grouped_dense(Ws, Ss, draws[0][6][0], draws[0][6][1], x, xs)
            row = {"projection": name, "M": M, "K": K, "tokens": tokens,
                   "distinct_experts": float(np.mean([d[4] for d in draws]))}
            for fmt, experts, f in formats:
                def launch(i):
                    ge, gb, xr, mx = draws[i][:4]
                    f(experts, ge, gb, xr, mx, xd, xsd, y=y, workspace=ws)

                launch(0)
                torch.cuda.synchronize()
                err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
                assert (err <= 1e-5 * mag).all(), f"bench: grouped {fmt} {name} tokens={tokens} disagrees with the oracle"
                us = graph_time_flushed_us(torch, stream, launch, len(draws), flush)
                # (the other bound: the same launches back to back without the flush, everything in L2)
                us_hot = graph_time_us(torch, stream, launch, len(draws))
                nbytes = float(np.mean([d[5][fmt] for d in draws]))
                row[fmt] = {"us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak, "bytes": nbytes,
                            "us_l2_resident": us_hot}
            row["speedup_vs_trit5"] = row["trit5"]["us"] / row["bitcos"]["us"]
            row["byte_ratio_trit5"] = row["trit5"]["bytes"] / row["bitcos"]["bytes"]
            row["speedup_vs_bit2"] = row["bit2"]["us"] / row["bitcos"]["us"]
            row["byte_ratio_bit2"] = row["bit2"]["bytes"] / row["bitcos"]["bytes"]
            out.append(row)
        del formats
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-detail", action="store_true", help="skip the per-shape / per-format table")
    ap.add_argument("--serial", action="store_true", help="launch the seven GEMVs of a step strictly in sequence")
    ap.add_argument("--branches", action="store_true",
                    help="seven launches per step with q|k|v and gate|up on parallel graph branches")
    ap.add_argument("--launch", default="multi", choices=["multi", "phased"],
                    help="multi: four bitcos_gemv_multi launches per step; phased: the whole layer pass as one "
                         "bitcos_gemv_phased launch (phases q|k|v, o, gate|up, down)")
    ap.add_argument("--no-prefetch", dest="prefetch", action="store_false",
                    help="plain bitcos_gemv_multi launches: no launch asks for the next launch's packed weights to be brought into L2")
    ap.add_argument("--no-chain-hint", dest="chain_hint", action="store_false",
                    help="launches are not told which launch runs directly before them (no uneven split between "
                         "thread blocks that start at once and thread blocks that start late)")
    ap.add_argument("--prefetch-launches", type=lambda v: [int(t) for t in v.split(",")], default=[1, 2],
                    help="with --prefetch: which of the step's four launches carry a request")
    ap.add_argument("--prefetch-depth", type=lambda v: [int(t) for t in v.split(",")], default=[1],
                    help="with --prefetch: which later launches' weights a launch asks for (1 = the next one)")
    ap.add_argument("--no-graph", action="store_true", help="plain stream launches instead of CUDA graphs (for profilers)")
    ap.add_argument("--e2e-per-phase", action="store_true",
                    help="end-to-end leg through four bitcos_gemv_multi_host calls per step instead of one bitcos_gemv_phases_host call")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle")
    ap.add_argument("--profile-quant", default="", choices=["", "chain", "fused"],
                    help="only launch --steps layer passes from bf16 activations (quantiser kernels in front of the "
                         "products, or inside them), without graphs (for profilers)")
    ap.add_argument("--profile-entry", default="gemv", choices=["gemv", "blend"],
                    help="entry point --profile-batch launches: bitcos_gemv or bitcos_gemv_blend_bf16")
    ap.add_argument("--profile-shape", default="8192x5120", metavar="MxK",
                    help="matrix of --profile-batch (default: the batch table's q projection)")
    ap.add_argument("--profile-batch", type=int, default=0, metavar="B",
                    help="only launch bitcos_gemv at batch B on the batch table's matrix, --steps times (for profilers)")
    ap.add_argument("--layer-only", action="store_true",
                    help="leave out the tables of the other configurations (density sweep, Qwen3-32B-shaped layer, experts)")
    ap.add_argument("--all-configs", action="store_true", help="add the device-side packing table")
    args = ap.parse_args()
    if args.profile_batch:
        if args.steps is None:
            args.steps = 6
        run_profile_batch(args)
        return
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 3
        run_reference(args)
    else:
        if args.steps is None:
            args.steps = 20 if args.profile_quant else 200
        run_cuda(args)


if __name__ == "__main__":
    main()
