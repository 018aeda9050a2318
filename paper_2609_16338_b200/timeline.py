"""Where a thread block of the layer pass spends its time: per-block time stamps from a debug build.

    python -m paper_2609_16338_b200.timeline [--no-prefetch] [--no-hint] [--steps 20]

Builds a second copy of the library with -DBITCOS_TIMELINE (libbitcos_timeline.so, next to the regular
one; the regular library carries no stamps), runs the BitNet-2B decoder layer as the benchmark does (four
bitcos_gemv_multi launches per step, rotated weight copies, one CUDA graph of `--steps` steps) and prints

  * for a few steps, when the first and the last block of each launch started and ended, and
  * per launch, the median [10 %, 90 %] over blocks and steps of each stamp, in nanoseconds from the block's
    first instruction, separately for blocks that found a free multiprocessor at once ("early") and blocks
    that had to wait for a block of the previous launch to leave ("late").

The stamps cost time (the instrumented pass is about 2 us slower than the regular one): read intervals and
order, not the total.  Stamps: clock64 of the stamping warp (producer warp's lane 0 up to "first copies out",
decoder warp 0 from "table arrived" to "decoders done", epilogue warp for the rest); launches are aligned
with each other through one globaltimer reading per block.
"""
from __future__ import annotations

import argparse
import ctypes as C
import os
import subprocess

import numpy as np

STAMPS = [  # (slot, label)
    (20, "arguments read"), (16, "layout worked out"), (13, "producer warp starts"), (14, "barriers initialised"),
    (15, "table requested"), (2, "at the block barrier (producer)"), (3, "table arrived (decoders)"),
    (4, "first stage arrived"), (5, "first tile decoded"), (6, "activations arrived"), (7, "first item's sums posted"),
    (8, "dependency resolved (epilogue)"), (10, "decoders done"), (9, "epilogue done"),
]
NAMES = ["q+k+v", "o", "gate+up", "down"]


def build_debug_library() -> str:
    from . import build
    path = os.path.join(build.HERE, "libbitcos_timeline.so")
    newest = max(os.path.getmtime(f) for f in build.SOURCES + build.HEADERS)
    if not os.path.exists(path) or os.path.getmtime(path) < newest:
        cmd = build.nvcc_command(("-DBITCOS_TIMELINE",))
        cmd[cmd.index("-o") + 1] = path
        subprocess.check_call(cmd)
    return path


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--no-prefetch", action="store_true", help="no launch asks for the next launch's weights")
    ap.add_argument("--no-hint", action="store_true", help="no launch is told which launch runs before it")
    ap.add_argument("--mhz", type=float, default=1965.0, help="SM clock the cycle counts are converted with")
    args = ap.parse_args()

    import torch
    import datagen
    from . import binding
    binding._LIB_PATH = build_debug_library()
    import paper_2609_16338_b200 as bc
    L = bc.load_library()
    L.bitcos_debug_timeline.argtypes = [C.c_void_p, C.c_int]
    L.bitcos_debug_timeline.restype = None

    cfg = datagen.CONFIG_BITNET_2B
    mats = []
    for i, (name, M, K) in enumerate(cfg["shapes"]):
        seed = datagen.config_seed(1, i)
        mats.append((M, K, bc.bitcos_pack(datagen.trits(seed, M, K, cfg["z"]), datagen.scales(seed, M, K)),
                     datagen.activations(seed, 1, K)))
    packed_bytes = sum(m[2].payload_bytes() for m in mats)
    copies = max(2, int(np.ceil(4.2 * 126e6 / packed_bytes)))
    base = [m[2].to_device() for m in mats]
    reps = [base] + [[w.clone() for w in base] for _ in range(copies - 1)]
    xs = [(torch.from_numpy(m[3][0]).cuda(), torch.from_numpy(m[3][1]).cuda()) for m in mats]
    ys = [torch.empty((1, m[0]), dtype=torch.float32, device="cuda") for m in mats]
    wss = [bc.make_workspace(m[0], m[1]) for m in mats]
    groups = [[0, 1, 2], [3], [4, 5], [6]]
    multi = [[bc.MultiJobs([(rep[j], xs[j][0], xs[j][1], ys[j], wss[j]) for j in g]) for g in groups] for rep in reps]
    nexts = [[bc.NextWeights([reps[c][j] for j in groups[(gi + 1) % 4]]) for gi in range(4)] for c in range(copies)]
    prevs = [bc.NextWeights([base[j] for j in groups[gi - 1]]) for gi in range(4)]

    def step(i):
        for gi, mj in enumerate(multi[i % copies]):
            bc.bitcos_gemv_multi(mj, next=nexts[i % copies][gi] if (not args.no_prefetch and gi in (1, 2)) else None,
                                 prev=None if args.no_hint else prevs[gi])

    slots = args.steps * 4
    tl = torch.zeros((slots, 160, 32), dtype=torch.int64, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(3):
            step(i)
        stream.synchronize()
        L.bitcos_debug_timeline(tl.data_ptr(), slots)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(args.steps):
                step(i)
        L.bitcos_debug_timeline(None, 1)
        for _ in range(5):
            g.replay()
        stream.synchronize()
        tl.zero_()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        g.replay()
        e1.record(stream)
        stream.synchronize()
    print(f"instrumented pass: {e0.elapsed_time(e1) * 1000 / args.steps:.2f} us per step")
    T = tl.cpu().numpy().astype(np.int64)

    def ns(cycles):
        return cycles / args.mhz * 1000.0

    # one globaltimer reading per block (slot 0, taken by the producer warp at slot 13's clock): block start in global time
    def starts_ends(t):
        used = t[:, 0] > 0
        t = t[used]
        start = t[:, 0] - ns(t[:, 13] - t[:, 1]).astype(np.int64)
        return start, t[:, 11], t

    first = None
    print("step  launch   blocks  first/last block start  first/last block end   (ns)")
    for st in range(args.steps // 2, min(args.steps // 2 + 4, args.steps)):
        for gi in range(4):
            s, e, _ = starts_ends(T[st * 4 + gi])
            first = s.min() if first is None else first
            print(f"{st:4d}  {NAMES[gi]:8s} {len(s):6d}  {s.min() - first:8d} {s.max() - first:8d}       {e.min() - first:8d} {e.max() - first:8d}")
    for gi in range(4):
        rows = {lab: ([], []) for _, lab in STAMPS}
        n_late = n_all = 0
        life = ([], [])
        for st in range(args.steps // 4, args.steps):
            s, e, t = starts_ends(T[st * 4 + gi])
            _, pe, _ = starts_ends(T[st * 4 + gi - 1])
            late = s > pe.min()          # started after the first block of the launch before had ended
            n_late += int(late.sum())
            n_all += len(late)
            for slot, lab in STAMPS:
                v = ns(t[:, slot] - t[:, 1])
                ok = t[:, slot] > 0
                rows[lab][0].extend(v[ok & ~late])
                rows[lab][1].extend(v[ok & late])
            life[0].extend((e - s)[~late])
            life[1].extend((e - s)[late])
        print(f"== {NAMES[gi]}: {n_all // (args.steps - args.steps // 4)} blocks per launch, {n_late / n_all:.2f} of them late")

        def fmt(z):
            return "       -" if len(z) == 0 else f"{np.median(z):7.0f} [{np.percentile(z, 10):6.0f}, {np.percentile(z, 90):6.0f}]"
        for _, lab in STAMPS:
            print(f"   {lab:34s} early {fmt(rows[lab][0])}    late {fmt(rows[lab][1])}")
        print(f"   {'block start to end (global timer)':34s} early {fmt(life[0])}    late {fmt(life[1])}")


if __name__ == "__main__":
    main()
