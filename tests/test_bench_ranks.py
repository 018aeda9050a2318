"""The benchmark's N > 1 path on CPU: two processes, gloo backend.

The product path does not shard and has no exchange step (independent replicas), so what several
ranks share is only the launcher contract: a barrier around the timed region, the maximum over the
ranks' times, whole-job aggregation, and one JSON line from rank 0 alone.
"""
import json
import os
import socket
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch(world, argv, extra_env=None):
    port = free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable] + argv, cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=600)
        outs.append((p.returncode, out, err))
    return outs


def test_ranks_barrier_and_max_over_two_gloo_processes(tmp_path):
    script = tmp_path / "ranks_probe.py"
    script.write_text(textwrap.dedent("""
        import json, sys, time
        sys.path.insert(0, %r)
        import bench
        r = bench.Ranks("gloo")
        assert r.world == 2
        # rank 1 is late for the barrier; both must leave it only after rank 1 arrived
        if r.rank == 1:
            time.sleep(0.5)
        t0 = time.time()
        r.barrier()
        left = time.time()
        # per-rank times differ; everybody gets the larger one
        mine = 10.0 + 5.0 * r.rank
        worst = r.max(mine)
        print(json.dumps({"rank": r.rank, "worst": worst, "left": left,
                          "value": bench.whole_job_value(worst, r.world)}))
        r.close()
    """ % ROOT))
    outs = launch(2, [str(script)])
    lines = []
    for rc, out, err in outs:
        assert rc == 0, err
        lines.append(json.loads(out.strip().splitlines()[-1]))
    lines.sort(key=lambda d: d["rank"])
    assert [d["worst"] for d in lines] == [15.0, 15.0]
    assert [d["value"] for d in lines] == [7.5, 7.5]          # two replicas: two tokens per step
    assert abs(lines[0]["left"] - lines[1]["left"]) < 0.4        # nobody left the barrier early


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    env = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK") if k in os.environ}
    try:
        r = bench.Ranks("gloo")
        assert (r.world, r.rank) == (1, 0)
        r.barrier()
        assert r.max(3.25) == 3.25
        r.close()
    finally:
        os.environ.update(env)


def test_reference_arm_under_two_ranks_prints_one_line_from_rank_zero():
    outs = launch(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"])
    (rc0, out0, err0), (rc1, out1, err1) = outs
    assert rc0 == 0, err0
    assert rc1 == 0, err1
    assert out1.strip() == ""                                    # rank 1: no work, no output
    line = json.loads(out0.strip().splitlines()[-1])
    assert line["impl"] == "reference"
    assert line["n_gpus"] == 2 and line["unit"] == "us" and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["value"] > 0


def test_roofline_traffic_comes_from_the_committed_ncu_summary():
    """bench.py takes roofline.traffic from the ncu summary under profiles/, not from a constant of its
    own: the summary must exist, carry the figure and the commit it was captured at, and the figure
    must agree with the step total the summary's own table prints."""
    import re
    import bench
    step, src = bench.ncu_traffic()
    assert step is not None, src
    assert "commit" in src
    with open(os.path.join(bench.ROOT, bench.TRAFFIC_PROFILE)) as f:
        text = f.read()
    m = re.search(r"\*\*step\*\*.*?\*\*([\d ]+)\*\* \| \*\*([\d ]+)\*\*", text)
    assert m, "the summary's table has no step row"
    assert int(m.group(1).replace(" ", "")) == step
    # traffic against algorithmic bytes: a little below 1 when the activations, outputs and the lookup table
    # (part of the algorithmic figure) are served from L2, above 1 if anything were fetched twice
    assert 0.97 <= step / int(m.group(2).replace(" ", "")) < 1.2
