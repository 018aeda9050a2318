"""Host logic of the multi launch's work split (no GPU): bitcos_gemv_multi_plan reproduces, block by block,
what bitcos_gemv_multi / bitcos_gemv_multi_chained would launch.  Whatever the shapes and the hint about the
launch before it, every item of every job is handed to exactly one thread block, no launch is larger than the
machine, and the uneven split only appears where it cannot touch a sum (rows that fit one item)."""
import numpy as np
import pytest

import paper_2609_16338_b200 as bc
from paper_2609_16338_b200 import build


@pytest.fixture(scope="module", autouse=True)
def library():
    build.build()
    bc.load_library()


def items_of_block(plan, b):
    """The items block b works on, from the plan's description of its walk."""
    j = plan["block"]["job"][b]
    first, n = plan["block"]["first_item"][b], plan["block"]["items"][b]
    cs, stride = plan["per_job"]["column_blocks"][j], plan["per_job"]["chunk_stride"][j]
    if stride == 1:
        return j, list(range(first, first + n))
    out, c, col = [], first // cs, first % cs
    for _ in range(n):
        out.append(c * cs + col)
        col += 1
        if col == cs:
            col, c = 0, c + stride
    return j, out


def check_cover(plan, n_jobs):
    seen = [dict() for _ in range(n_jobs)]
    for b in range(plan["n_blocks"]):
        j, its = items_of_block(plan, b)
        for i in its:
            assert i not in seen[j], f"item {i} of job {j} handed out twice"
            seen[j][i] = b
    for j in range(n_jobs):
        assert sorted(seen[j]) == list(range(plan["per_job"]["items"][j])), f"job {j}: items missing"


LAYER = {"q+k+v": [(2560, 2560), (640, 2560), (640, 2560)], "o": [(2560, 2560)],
         "gate+up": [(6912, 2560), (6912, 2560)], "down": [(2560, 6912)]}


def test_layer_launches_as_documented():
    sms = 148
    grid = {k: bc.bitcos_gemv_multi_plan(v, 1, sms)["n_blocks"] for k, v in LAYER.items()}
    # two consecutive small launches fit side by side; the launch with no more items than the other leaves free
    # runs one item per block
    assert grid["q+k+v"] <= sms * 46 // 100 and grid["o"] == 80 and grid["q+k+v"] + grid["o"] <= sms
    assert grid["gate+up"] == sms and grid["down"] == 80
    # gate+up told that o's 80 blocks run before it: 68 blocks start at once and take four items, 80 take two
    p = bc.bitcos_gemv_multi_plan(LAYER["gate+up"], 1, sms, grid["o"])
    check_cover(p, 2)
    early, late = p["block"]["items"][:sms - grid["o"]], p["block"]["items"][sms - grid["o"]:]
    assert set(early) == {4} and set(late) == {2}
    # both jobs have early blocks and late blocks
    assert set(p["block"]["job"][:sms - grid["o"]]) == {0, 1} and set(p["block"]["job"][sms - grid["o"]:]) == {0, 1}
    # down (rows cut into three column blocks) is never split unevenly, whatever it is told
    for busy in (0, 40, 80, 148):
        q = bc.bitcos_gemv_multi_plan(LAYER["down"], 1, sms, busy)
        check_cover(q, 1)
        assert set(q["block"]["items"]) == {3} and q["per_job"]["column_blocks"] == [3]
    # launches that start entirely early or entirely late are split evenly
    for name, busy in (("q+k+v", grid["down"]), ("o", grid["q+k+v"]), ("gate+up", 0), ("gate+up", sms), ("gate+up", 200)):
        q = bc.bitcos_gemv_multi_plan(LAYER[name], 1, sms, busy)
        check_cover(q, len(LAYER[name]))
        assert max(q["block"]["items"]) - min(q["block"]["items"]) <= 1, (name, busy)


@pytest.mark.parametrize("seed", range(40))
def test_every_item_once_for_random_launches(seed):
    rng = np.random.default_rng(1000 + seed)
    n_jobs = int(rng.integers(1, 9))
    shapes = [(int(rng.integers(1, 9000)), 128 * int(rng.integers(1, 80))) for _ in range(n_jobs)]
    batch = int(rng.choice([1, 2, 3, 8, 16]))
    sms = int(rng.choice([148, 132, 20, 160]))
    busy = int(rng.choice([0, 1, sms // 3, sms // 2, sms - 1, sms, 3 * sms]))
    p = bc.bitcos_gemv_multi_plan(shapes, batch, sms, busy)
    assert 1 <= p["n_blocks"] <= max(sms, n_jobs)         # (every job gets at least one block)
    check_cover(p, n_jobs)
    uneven = max(p["block"]["items"]) - min(p["block"]["items"]) > 1 and len(set(p["block"]["job"])) == 1
    if uneven and 0 < busy < sms:
        assert all(cs == 1 for cs in p["per_job"]["column_blocks"])
    # the same launch without the hint hands out the same items
    q = bc.bitcos_gemv_multi_plan(shapes, batch, sms, 0)
    check_cover(q, n_jobs)
    assert q["per_job"]["items"] == p["per_job"]["items"] and q["n_blocks"] == p["n_blocks"]


def test_malformed_requests_are_refused():
    L = bc.load_library()
    with pytest.raises(RuntimeError):
        bc.bitcos_gemv_multi_plan([(32, 100)], 1, 148, 0)              # K not a multiple of 128
    with pytest.raises(RuntimeError):
        bc.bitcos_gemv_multi_plan([(32, 128)] * 9, 1, 148, 0)          # more jobs than a launch takes
    with pytest.raises(RuntimeError):
        bc.bitcos_gemv_multi_plan([(32, 128)], 17, 148, 0)
    with pytest.raises(RuntimeError):
        bc.bitcos_gemv_multi_plan([(32, 128)], 1, 0, 0)
    assert L.bitcos_gemv_multi_plan(None, None, 1, 1, 148, 0, 0, None, None, None, None, None, None, None, None) != 0
