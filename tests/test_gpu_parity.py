"""GPU parity: every device entry point of the C ABI against the CPU oracle, element by
element, on the same seeded inputs.

Bar: int32 group accumulators bit-exact; fp32 outputs within 1e-5 of sum|terms|
(|y - y_ref| <= 1e-5 * mag, and exactly 0 where mag is 0).
"""
import numpy as np
import pytest

import datagen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL = 1e-5


@pytest.fixture(scope="module")
def bc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_16338_b200 as m
    from paper_2609_16338_b200 import build
    build.build()
    m.load_library()
    return m


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def check(y, acc, acc_ref, y_ref, mag, what):
    torch.cuda.synchronize()
    if acc is not None:
        assert np.array_equal(acc.cpu().numpy(), acc_ref), f"{what}: int32 accumulators differ"
    yv = y.cpu().numpy().astype(np.float64)
    err = np.abs(yv - y_ref)
    bad = err > REL * mag
    assert not bad.any(), f"{what}: {bad.sum()} outputs off, worst {np.max(err / np.maximum(mag, 1e-300)):.3e}"
    assert (yv[mag == 0] == 0).all()


def run_all_formats(bc, W, S, x, xs, what, formats=("bitcos", "trit5", "bit2"), debug=True):
    M, K = W.shape
    acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
    xd, xsd = dev(x), dev(xs)
    ws = bc.make_workspace(M, K)
    st = bc.scales_tile(S, M, K)
    for fmt in formats:
        if fmt == "bitcos":
            Wd = bc.bitcos_pack(W, S).to_device()
            f = bc.bitcos_gemv
        elif fmt == "trit5":
            Wd = bc.plain_to_device(bc.trit5_pack(W), st, M, K)
            f = bc.trit5_gemv
        else:
            Wd = bc.plain_to_device(bc.bit2_pack(W), st, M, K)
            f = bc.bit2_gemv
        for rep in range(2):                          # twice: the workspace must come back clean
            y, acc = f(Wd, xd, xsd, acc_debug=debug if rep == 0 else None, workspace=ws)
            check(y, acc, acc_ref, y_ref, mag, f"{what} {fmt} rep{rep}")
    return acc_ref, y_ref, mag


def test_config0_tiny(bc):
    M, K, z = 256, 512, 0.42
    s = datagen.config_seed(0, 0)
    W, S = datagen.trits(s, M, K, z), datagen.scales(s, M, K)
    x, xs = datagen.activations(s, 1, K)
    run_all_formats(bc, W, S, x, xs, "config0")


@pytest.mark.parametrize("M,K,B", [
    (32, 128, 1), (1, 128, 1), (33, 256, 2), (100, 384, 3), (640, 2560, 1), (96, 6912, 1), (64, 2176, 5),
    (256, 512, 16), (50, 1280, 8), (2560, 2560, 1), (160, 25600, 2), (320, 8192, 1),
    # four tokens and more: the contraction runs on the tensor cores; rows in one piece (K <= 2560,
    # or 2048 for more than eight tokens) and rows cut into column blocks
    (96, 6912, 8), (64, 5120, 16), (40, 3072, 4), (2560, 2560, 16), (33, 2560, 9), (700, 2048, 12), (65, 128, 7),
])
def test_shapes_and_batches(bc, M, K, B):
    W, S = datagen.trits(100 + M, M, K, 0.42), datagen.scales(100 + M, M, K)
    x, xs = datagen.activations(100 + K, B, K)
    run_all_formats(bc, W, S, x, xs, f"{M}x{K} B{B}")


def test_degenerate_weights_and_activations(bc):
    M, K = 96, 512
    S = datagen.scales(7, M, K)
    x, xs = datagen.activations(7, 2, K)
    x[0, :] = -128                                       # the int8 minimum is accepted
    x[1, ::2] = 127
    for fill in (0, 1, -1):
        run_all_formats(bc, np.full((M, K), fill, np.int8), S, x, xs, f"fill {fill}")
    W = np.zeros((M, K), np.int8)
    for k in (0, 31, 32, 127, 128, K - 1):
        W[:] = 0
        W[5, k] = -1
        W[37, k] = 1
        run_all_formats(bc, W, S, x, xs, f"single nonzero k={k}")
    # all scales one, activation scale one: y is an exact integer
    ones = np.full((M, K // 128), 0x3F80, np.uint16)
    W = datagen.trits(8, M, K, 0.3)
    acc_ref, y_ref, _ = run_all_formats(bc, W, ones, x, np.ones(2, np.float32), "unit scales")
    assert np.array_equal(y_ref, acc_ref.sum(-1).astype(np.float64))
    # dense rows next to empty rows (sign cursors far apart inside one tile)
    W = np.zeros((M, K), np.int8)
    W[::2] = datagen.trits(9, M // 2, K, 0.0)
    run_all_formats(bc, W, S, x, xs, "alternating dense / empty rows")


@pytest.mark.parametrize("z", [0.30, 0.375, 0.42, 0.47, 0.515])
def test_density_sweep_small(bc, z):
    M, K = 384, 1536
    W, S = datagen.trits(11, M, K, z), datagen.scales(11, M, K)
    x, xs = datagen.activations(11, 1, K)
    run_all_formats(bc, W, S, x, xs, f"z={z}")


def test_grouped_experts(bc):
    E, M, K, top_k = 16, 768, 2048, 4
    z = 0.3288
    Ws = [datagen.trits(200 + e, M, K, z) for e in range(E)]
    Ss = [datagen.scales(200 + e, M, K) for e in range(E)]
    experts = bc.DeviceExperts([bc.bitcos_pack(Ws[e], Ss[e]).to_device() for e in range(E)])
    for tokens in (1, 3, 16):
        x, xs = datagen.activations(300 + tokens, tokens, K)
        ids = datagen.expert_choices(300 + tokens, tokens, E, top_k)
        pair_expert = ids.reshape(-1)
        pair_xrow = np.repeat(np.arange(tokens, dtype=np.int32), top_k)
        order, ge, gb, xr, mx = bc.group_pairs(pair_expert, pair_xrow)
        acc_ref, y_ref, mag = oracle.grouped_dense(Ws, Ss, pair_expert[order], pair_xrow[order], x, xs)
        ws = bc.make_workspace(M, K, copies=len(ge))
        for rep in range(2):
            y, acc = bc.bitcos_gemv_grouped(experts, dev(ge), dev(gb), dev(xr), mx, dev(x), dev(xs),
                                            acc_debug=True, workspace=ws)
            check(y, acc, acc_ref, y_ref, mag, f"grouped tokens={tokens} rep{rep}")


def test_grouped_many_small_groups(bc):
    """More items than thread blocks and few items per group: blocks run the tail of one group and
    the head of the next (and whole small groups) without stopping their pipeline."""
    E, M, K, top_k = 96, 160, 1280, 6
    Ws = [datagen.trits(900 + e, M, K, 0.35) for e in range(E)]
    Ss = [datagen.scales(900 + e, M, K) for e in range(E)]
    experts = bc.DeviceExperts([bc.bitcos_pack(Ws[e], Ss[e]).to_device() for e in range(E)])
    for tokens in (16, 12):
        x, xs = datagen.activations(950 + tokens, tokens, K)
        ids = datagen.expert_choices(950 + tokens, tokens, E, top_k)
        pair_expert = ids.reshape(-1)
        pair_xrow = np.repeat(np.arange(tokens, dtype=np.int32), top_k)
        order, ge, gb, xr, mx = bc.group_pairs(pair_expert, pair_xrow)
        assert len(ge) * ((M + 31) // 32 + 1) // 2 > 148 or len(ge) > 50
        acc_ref, y_ref, mag = oracle.grouped_dense(Ws, Ss, pair_expert[order], pair_xrow[order], x, xs)
        ws = bc.make_workspace(M, K, copies=len(ge))
        for rep in range(2):
            y, acc = bc.bitcos_gemv_grouped(experts, dev(ge), dev(gb), dev(xr), mx, dev(x), dev(xs),
                                            acc_debug=True, workspace=ws)
            check(y, acc, acc_ref, y_ref, mag, f"many groups tokens={tokens} rep{rep}")


def test_grouped_malformed_routing_lists_are_skipped(bc):
    """Routing lists come from device memory (a router's output) and are checked on the device: a
    group that points outside the pair list, holds more pairs than the launch was sized for, names
    an expert or an activation row that does not exist is skipped whole -- its outputs keep what
    they held -- and the status word reads 2; the well-formed groups of the same call are right."""
    E, M, K, tokens = 6, 96, 512, 4
    Ws = [datagen.trits(1700 + e, M, K, 0.33) for e in range(E)]
    Ss = [datagen.scales(1700 + e, M, K) for e in range(E)]
    experts = bc.DeviceExperts([bc.bitcos_pack(Ws[e], Ss[e]).to_device() for e in range(E)])
    x, xs = datagen.activations(1700, tokens, K)
    pair_expert = np.array([0, 0, 2, 3, 3, 5], np.int32)
    pair_xrow = np.array([0, 1, 2, 0, 3, 1], np.int32)
    order, ge, gb, xr, mx = bc.group_pairs(pair_expert, pair_xrow)
    acc_ref, y_ref, mag = oracle.grouped_dense(Ws, Ss, pair_expert[order], pair_xrow[order], x, xs)
    n_groups = len(ge)

    def run(ge_, gb_, xr_, mx_, bad_group):
        ws = bc.make_workspace(M, K, copies=n_groups)
        y = torch.full((len(xr_), M), 777.0, dtype=torch.float32, device="cuda")
        y, _ = bc.bitcos_gemv_grouped(experts, dev(ge_), dev(gb_), dev(xr_), mx_, dev(x), dev(xs), y=y, workspace=ws)
        torch.cuda.synchronize()
        yh = y.cpu().numpy().astype(np.float64)
        for g in range(n_groups):
            rows = range(gb[g], gb[g + 1])
            for r in rows:
                if g in bad_group:
                    assert (yh[r] == 777.0).all(), ("skipped group was written", g)
                else:
                    assert (np.abs(yh[r] - y_ref[r]) <= REL * mag[r]).all(), ("good group wrong", g)
        assert bc.workspace_status(ws) == (2 if bad_group else 0)

    run(ge, gb, xr, mx, set())
    bad = ge.copy(); bad[1] = E + 3                    # an expert that does not exist
    run(bad, gb, xr, mx, {1})
    bad = ge.copy(); bad[2] = -1
    run(bad, gb, xr, mx, {2})
    bad = xr.copy(); bad[gb[0]] = tokens               # an activation row past the end of x
    run(ge, gb, bad, mx, {0})
    bad = xr.copy(); bad[gb[3]] = -5
    run(ge, gb, bad, mx, {3})
    run(ge, gb, xr, 1, {0, 2})                         # groups 0 and 2 hold two pairs, the launch was sized for one


def test_routing_grouped_on_the_device(bc):
    """The pairs stay on the device: bitcos_group_pairs_device sorts them by expert (stable), and
    bitcos_gemv_grouped_lists reads the number of groups from device memory.  Same lists as the host
    grouping, same outputs as the oracle; rows cut into column blocks (K = 6912) and rows in one piece."""
    for (E, M, K, top_k, tokens) in ((32, 160, 1280, 4, 5), (16, 96, 6912, 3, 2), (128, 768, 2048, 8, 16), (8, 64, 256, 2, 1)):
        Ws = [datagen.trits(1800 + e, M, K, 0.33) for e in range(E)]
        Ss = [datagen.scales(1800 + e, M, K) for e in range(E)]
        experts = bc.DeviceExperts([bc.bitcos_pack(Ws[e], Ss[e]).to_device() for e in range(E)])
        x, xs = datagen.activations(1800 + tokens, tokens, K)
        ids = datagen.expert_choices(1800 + tokens, tokens, E, top_k)
        rng = np.random.default_rng(E)
        perm = rng.permutation(tokens * top_k)                     # pairs in no particular order
        pair_expert = ids.reshape(-1)[perm].astype(np.int32)
        pair_xrow = np.repeat(np.arange(tokens, dtype=np.int32), top_k)[perm]
        order_h, ge_h, gb_h, xr_h, mx = bc.group_pairs(pair_expert, pair_xrow)
        ge, gb, xr, order, ng = bc.bitcos_group_pairs_device(dev(pair_expert), dev(pair_xrow), E)
        torch.cuda.synchronize()
        n = int(ng.item())
        assert n == len(ge_h)
        assert np.array_equal(ge.cpu().numpy()[:n], ge_h) and np.array_equal(gb.cpu().numpy()[:n + 1], gb_h)
        assert np.array_equal(xr.cpu().numpy(), xr_h) and np.array_equal(order.cpu().numpy(), order_h)
        acc_ref, y_ref, mag = oracle.grouped_dense(Ws, Ss, pair_expert[order_h], pair_xrow[order_h], x, xs)
        for rep in range(2):
            y, acc = bc.bitcos_gemv_grouped_lists(experts, ge, gb, ng, xr, min(tokens, 16), dev(x), dev(xs), acc_debug=True)
            check(y, acc, acc_ref, y_ref, mag, f"device routing E={E} tokens={tokens} rep{rep}")


def test_grouped_down_projection_shape(bc):
    # K = 768 (six groups), per-pair activation rows
    E, M, K = 4, 2048, 768
    Ws = [datagen.trits(400 + e, M, K, 0.3288) for e in range(E)]
    Ss = [datagen.scales(400 + e, M, K) for e in range(E)]
    experts = bc.DeviceExperts([bc.bitcos_pack(Ws[e], Ss[e]).to_device() for e in range(E)])
    pair_expert = np.array([3, 0, 3, 1, 0, 3], np.int32)
    pair_xrow = np.arange(6, dtype=np.int32)
    x, xs = datagen.activations(401, 6, K)
    order, ge, gb, xr, mx = bc.group_pairs(pair_expert, pair_xrow)
    acc_ref, y_ref, mag = oracle.grouped_dense(Ws, Ss, pair_expert[order], pair_xrow[order], x, xs)
    y, acc = bc.bitcos_gemv_grouped(experts, dev(ge), dev(gb), dev(xr), mx, dev(x), dev(xs), acc_debug=True)
    check(y, acc, acc_ref, y_ref, mag, "grouped down")


@pytest.mark.parametrize("B", [1, 3])
def test_multi_launch_matches_separate_products(bc, B):
    """Several independent matrices (different shapes, also different K) in one launch."""
    shapes = [(2560, 2560), (640, 2560), (96, 6912), (320, 1280), (64, 128), (33, 2560), (1000, 512), (32, 5120)]
    jobs, refs = [], []
    for i, (M, K) in enumerate(shapes):
        W, S = datagen.trits(600 + i, M, K, 0.4219), datagen.scales(600 + i, M, K)
        x, xs = datagen.activations(600 + i, B, K)
        refs.append(oracle.gemv_dense(W, S, x, xs))
        y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
        jobs.append((bc.bitcos_pack(W, S).to_device(), dev(x), dev(xs), y, bc.make_workspace(M, K)))
    for n in (8, 5, 3, 1):
        for rep in range(2):
            for j in jobs:
                j[3].fill_(float("nan"))
            bc.bitcos_gemv_multi(jobs[:n])
            for (Wd, _, _, y, _), (acc_ref, y_ref, mag) in zip(jobs[:n], refs[:n]):
                check(y, None, acc_ref, y_ref, mag, f"multi n={n} rep{rep} {Wd.M}x{Wd.K}")
    # the same results as the single-matrix entry point, bit for bit
    bc.bitcos_gemv_multi(jobs)
    torch.cuda.synchronize()
    for (Wd, x, xs, y, ws) in jobs:
        y1, _ = bc.bitcos_gemv(Wd, x, xs, workspace=ws)
        torch.cuda.synchronize()
        assert torch.equal(y1, y)


def test_multi_launch_with_l2_request_for_later_matrices(bc):
    """bitcos_gemv_multi_chained, `next`: the launch also asks for other matrices' packed arrays to be brought into
    L2.  Whatever `next` holds (large, tiny, without the host copy of the entry offsets, the launch's own
    matrices, seven entries), the results are those of the oracle and of bitcos_gemv_multi bit for bit; a
    malformed `next` is refused before anything is launched."""
    shapes = [(2560, 2560), (640, 2560), (96, 6912), (33, 256)]
    jobs, refs, plain = [], [], []
    for i, (M, K) in enumerate(shapes):
        W, S = datagen.trits(650 + i, M, K, 0.4219), datagen.scales(650 + i, M, K)
        x, xs = datagen.activations(650 + i, 1, K)
        refs.append(oracle.gemv_dense(W, S, x, xs))
        y = torch.full((1, M), float("nan"), dtype=torch.float32, device="cuda")
        jobs.append((bc.bitcos_pack(W, S).to_device(), dev(x), dev(xs), y, bc.make_workspace(M, K)))
    bc.bitcos_gemv_multi(jobs)
    torch.cuda.synchronize()
    plain = [j[3].clone() for j in jobs]
    later = [bc.bitcos_pack(datagen.trits(660 + i, M, K, 0.4219), datagen.scales(660 + i, M, K)).to_device()
             for i, (M, K) in enumerate([(6912, 2560), (2560, 6912), (32, 128), (70, 384)])]
    nexts = [later[:1], later, [w.without_host_offsets() for w in later], [j[0] for j in jobs],
             (later + later)[:7], []]
    for n_jobs in (4, 1):
        for nx in nexts:
            for j in jobs:
                j[3].fill_(float("nan"))
            bc.bitcos_gemv_multi(jobs[:n_jobs], next=nx)
            for (Wd, _, _, y, ws), (acc_ref, y_ref, mag), y0 in zip(jobs[:n_jobs], refs, plain):
                check(y, None, acc_ref, y_ref, mag, f"prefetch {len(nx)} later matrices, {Wd.M}x{Wd.K}")
                assert torch.equal(y, y0)
                assert bc.workspace_status(ws) == 0
    # a following product reads what was requested: still the oracle's numbers
    M, K = 6912, 2560
    W, S = datagen.trits(660, M, K, 0.4219), datagen.scales(660, M, K)
    x, xs = datagen.activations(670, 1, K)
    bc.bitcos_gemv_multi(jobs, next=later[:1])
    y, acc = bc.bitcos_gemv(later[0], dev(x), dev(xs), acc_debug=True)
    check(y, acc, *oracle.gemv_dense(W, S, x, xs), "product after the request")
    with pytest.raises(RuntimeError):
        bc.bitcos_gemv_multi(jobs, next=(later + later))         # eight entries: more than the launch carries
    L = bc.load_library()
    mj = bc.MultiJobs(jobs)
    assert L.bitcos_gemv_multi_chained(mj.arr, len(mj.arr), 1, None, 0, None, 1, None) != 0
    assert L.bitcos_gemv_multi_chained(mj.arr, len(mj.arr), 1, None, 1, None, 0, None) != 0


def test_multi_launch_told_what_runs_before_it(bc):
    """bitcos_gemv_multi_chained, `prev`: the launch hands the blocks it expects to start at once more work items
    than the ones it expects to start late, and interleaves the jobs' blocks.  Every output still matches the
    oracle and bitcos_gemv_multi bit for bit: for previous launches of every size (a few blocks, about half the
    chip -- the case that changes the split --, the whole chip), for jobs whose rows are cut into column blocks
    (hint not applied) and for jobs with fewer items than blocks."""
    cases = {
        "gate+up": [(6912, 2560), (6912, 2560)],
        "three": [(2560, 2560), (4000, 2560), (1333, 1280)],
        "cut rows": [(2560, 6912), (2560, 2560)],
        "small": [(640, 2560), (96, 128)],
    }
    prevs = {"few blocks": [(320, 2560)], "half the chip": [(2560, 2560)], "more than half": [(3000, 2560)],
             "whole chip": [(6912, 2560), (6912, 2560)], "tiny": [(32, 128)]}
    prev_w = {k: [bc.bitcos_pack(datagen.trits(690 + i, M, K, 0.4219), datagen.scales(690 + i, M, K)).to_device()
                  for i, (M, K) in enumerate(v)] for k, v in prevs.items()}
    for name, shapes in cases.items():
        for B in (1, 2, 5):
            jobs, refs = [], []
            for i, (M, K) in enumerate(shapes):
                W, S = datagen.trits(680 + i, M, K, 0.4219), datagen.scales(680 + i, M, K)
                x, xs = datagen.activations(680 + i + 10 * B, B, K)
                refs.append(oracle.gemv_dense(W, S, x, xs))
                y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
                jobs.append((bc.bitcos_pack(W, S).to_device(), dev(x), dev(xs), y, bc.make_workspace(M, K)))
            bc.bitcos_gemv_multi(jobs)
            torch.cuda.synchronize()
            plain = [j[3].clone() for j in jobs]
            for pname, pw in prev_w.items():
                for rep in range(2):
                    for j in jobs:
                        j[3].fill_(float("nan"))
                    bc.bitcos_gemv_multi(jobs, prev=pw, next=[jobs[0][0]] if rep else None)
                    for (Wd, _, _, y, ws), (acc_ref, y_ref, mag), y0 in zip(jobs, refs, plain):
                        check(y, None, acc_ref, y_ref, mag, f"{name} B={B} after {pname}, {Wd.M}x{Wd.K}")
                        assert torch.equal(y, y0), f"{name} B={B} after {pname}"
                        assert bc.workspace_status(ws) == 0


@pytest.mark.parametrize("B", [1, 2, 3])
def test_multi_launch_recorded_into_a_graph(bc, B):
    """Recorded into a CUDA graph, a multi launch of one or two tokens carries a host-made table of every
    block's first copies, which the kernel issues with its first instructions (a plain stream launch goes
    without it).  Replayed, the outputs are those of the oracle and of the plain launch bit for bit: layer
    shapes, ragged row counts, rows cut into column blocks, a job with a single tile, jobs with and
    without the host copy of the entry offsets, with and without the sequence hints, several replays."""
    sets = {
        "gate+up": [(6912, 2560), (6912, 2560)],
        "q+k+v": [(2560, 2560), (640, 2560), (640, 2560)],
        "down": [(2560, 6912)],
        "ragged": [(1000, 512), (33, 2560), (32, 128), (70, 384)],
        "two tiles per warp": [(25600, 2560), (12000, 2560)],
    }
    side = torch.cuda.Stream()
    for name, shapes in sets.items():
        jobs, refs = [], []
        for i, (M, K) in enumerate(shapes):
            W, S = datagen.trits(720 + i, M, K, 0.4219), datagen.scales(720 + i, M, K)
            x, xs = datagen.activations(720 + i + 10 * B, B, K)
            refs.append(oracle.gemv_dense(W, S, x, xs))
            y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
            Wd = bc.bitcos_pack(W, S).to_device()
            jobs.append((Wd, dev(x), dev(xs), y, bc.make_workspace(M, K)))
        bc.bitcos_gemv_multi(jobs)
        torch.cuda.synchronize()
        plain = [j[3].clone() for j in jobs]
        variants = [("no hints", jobs, None, None), ("hints", jobs, [jobs[0][0]], [jobs[-1][0]])]
        if name == "ragged":
            mixed = [(j[0].without_host_offsets() if i == 1 else j[0],) + j[1:] for i, j in enumerate(jobs)]
            variants.append(("one job without host offsets", mixed, None, None))
        for tag, js, prev, nxt in variants:
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    bc.bitcos_gemv_multi(js, prev=prev, next=nxt)
                for rep in range(3):
                    for j in jobs:
                        j[3].fill_(float("nan"))
                    g.replay()
                    side.synchronize()
                    for (Wd, _, _, y, ws), (acc_ref, y_ref, mag), y0 in zip(jobs, refs, plain):
                        check(y, None, acc_ref, y_ref, mag, f"recorded {name} B={B} {tag} rep{rep} {Wd.M}x{Wd.K}")
                        assert torch.equal(y, y0), f"recorded {name} B={B} {tag} rep{rep}"
                        assert bc.workspace_status(ws) == 0
            del g


@pytest.mark.parametrize("B", [1, 2])
def test_single_launches_recorded_into_a_graph(bc, B):
    """The single-matrix products of all three formats recorded into a CUDA graph, two launches back to back (the
    second starts under the first): accumulators bit for bit, outputs as the plain launch.  Layer shapes, ragged row counts, rows cut into column blocks (K = 6912, 12288), a single
    tile, BITCOS with and without the host copy of the entry offsets."""
    side = torch.cuda.Stream()
    for (M, K) in ((2560, 2560), (640, 2560), (2560, 6912), (1000, 512), (33, 12288), (32, 128), (70, 384), (4096, 1280)):
        W, S = datagen.trits(760 + M, M, K, 0.4219), datagen.scales(760 + M, M, K)
        x, xs = datagen.activations(760 + K + B, B, K)
        acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        st = bc.scales_tile(S, M, K)
        Wb = bc.bitcos_pack(W, S).to_device()
        cases = [("bitcos", Wb, bc.bitcos_gemv), ("bitcos without host offsets", Wb.without_host_offsets(), bc.bitcos_gemv),
                 ("trit5", bc.plain_to_device(bc.trit5_pack(W), st, M, K), bc.trit5_gemv),
                 ("bit2", bc.plain_to_device(bc.bit2_pack(W), st, M, K), bc.bit2_gemv)]
        ws = bc.make_workspace(M, K)
        for fmt, Wd, f in cases:
            y0, _ = f(Wd, xd, xsd, workspace=ws)
            torch.cuda.synchronize()
            y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
            acc = torch.full((B, M, K // 128), -1, dtype=torch.int32, device="cuda")
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    f(Wd, xd, xsd, y=y, acc_debug=acc, workspace=ws)
                    f(Wd, xd, xsd, y=y, acc_debug=acc, workspace=ws)      # twice in a row: the second starts under the first
                for rep in range(2):
                    y.fill_(float("nan"))
                    acc.fill_(-1)
                    g.replay()
                    side.synchronize()
                    check(y, acc, acc_ref, y_ref, mag, f"recorded {fmt} {M}x{K} B={B} rep{rep}")
                    assert torch.equal(y, y0), f"recorded {fmt} {M}x{K} B={B}"
                    assert bc.workspace_status(ws) == 0
            del g


def test_recorded_chained_launches_random(bc):
    """Sixty random multi launches (one to five jobs of mixed shapes, one to three tokens, random `prev` and `next`
    lists) recorded into CUDA graphs: every output bit for bit that of the plain single-matrix product, which the
    other tests hold against the oracle."""
    rng = np.random.default_rng(7)
    side = torch.cuda.Stream()
    pool = {}

    def mat(M, K):
        if (M, K) not in pool:
            z = float(rng.choice([0.3, 0.4219, 0.6]))
            pool[(M, K)] = bc.bitcos_pack(datagen.trits(M * 7 + K, M, K, z), datagen.scales(M + K, M, K)).to_device()
        return pool[(M, K)]

    Ms, Ks = [32, 33, 640, 1000, 2560, 4000, 6912, 70], [128, 384, 1280, 2560, 5120, 6912]
    for it in range(60):
        n, B = int(rng.integers(1, 6)), int(rng.choice([1, 2, 3]))
        jobs, plain = [], []
        for _ in range(n):
            Wd = mat(int(rng.choice(Ms)), int(rng.choice(Ks)))
            x, xs = datagen.activations(it * 10 + Wd.M + Wd.K, B, Wd.K)
            xd, xsd, ws = dev(x), dev(xs), bc.make_workspace(Wd.M, Wd.K)
            y0, _ = bc.bitcos_gemv(Wd, xd, xsd, workspace=ws)
            jobs.append((Wd, xd, xsd, torch.full((B, Wd.M), float("nan"), dtype=torch.float32, device="cuda"), ws))
            plain.append(y0)
        torch.cuda.synchronize()
        prev = [mat(int(rng.choice(Ms)), int(rng.choice(Ks))) for _ in range(int(rng.integers(0, 4)))] or None
        nxt = [mat(int(rng.choice(Ms)), int(rng.choice(Ks))) for _ in range(int(rng.integers(0, 4)))] or None
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                bc.bitcos_gemv_multi(jobs, prev=prev, next=nxt)
            g.replay()
            side.synchronize()
        for (Wd, _, _, y, ws), y0 in zip(jobs, plain):
            assert torch.equal(y, y0), (it, [(j[0].M, j[0].K) for j in jobs], B)
            assert bc.workspace_status(ws) == 0
        del g


def test_host_copy_of_entry_offsets_changes_nothing(bc):
    """With a host copy of tile_off the launch passes each block's first entry offsets by value;
    without it the kernel loads them.  Same results, bit for bit, and both match the oracle."""
    for (M, K, B) in ((2560, 2560, 1), (640, 6912, 1), (6912, 2560, 3), (96, 25600, 1)):
        W, S = datagen.trits(700 + M, M, K, 0.4219), datagen.scales(700 + M, M, K)
        x, xs = datagen.activations(700 + K, B, K)
        acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
        Wd = bc.bitcos_pack(W, S).to_device()
        assert Wd.tile_off_host is not None
        Wn = Wd.without_host_offsets()
        xd, xsd = dev(x), dev(xs)
        ws = bc.make_workspace(M, K)
        y1, acc1 = bc.bitcos_gemv(Wd, xd, xsd, acc_debug=True, workspace=ws)
        check(y1, acc1, acc_ref, y_ref, mag, f"host offsets {M}x{K}")
        y2, acc2 = bc.bitcos_gemv(Wn, xd, xsd, acc_debug=True, workspace=ws)
        check(y2, acc2, acc_ref, y_ref, mag, f"device offsets {M}x{K}")
        assert torch.equal(y1, y2)
        # one job with, one without: the launch falls back to loading them
        ya = torch.empty_like(y1)
        yb = torch.empty_like(y1)
        bc.bitcos_gemv_multi([(Wd, xd, xsd, ya, ws), (Wn, xd, xsd, yb, bc.make_workspace(M, K))])
        torch.cuda.synchronize()
        assert torch.equal(ya, y1) and torch.equal(yb, y1)


def test_host_buffer_entry_point(bc):
    M, K, B = 640, 2560, 4
    W, S = datagen.trits(21, M, K, 0.4219), datagen.scales(21, M, K)
    x, xs = datagen.activations(21, B, K)
    acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
    Wd = bc.bitcos_pack(W, S).to_device()
    staging = torch.empty(bc.bitcos_gemv_host_staging_bytes(M, K, B), dtype=torch.uint8, device="cuda")
    ws = bc.make_workspace(M, K)
    xh = torch.from_numpy(x).pin_memory()
    xsh = torch.from_numpy(xs).pin_memory()
    yh = torch.empty((B, M), dtype=torch.float32).pin_memory()
    bc.bitcos_gemv_host(Wd, xh.numpy(), xsh.numpy(), yh.numpy(), staging, ws)
    err = np.abs(yh.numpy().astype(np.float64) - y_ref)
    assert (err <= REL * mag).all()


def test_two_tiles_per_warp_every_output(bc):
    """Matrices large enough for the plan with two tiles per decoder warp (eight or more items per
    multiprocessor): whole rows in one item (K = 2560 and 5120) and rows cut in two column blocks
    (K = 6912); one and two tokens; all three formats.  Every accumulator and every output is
    compared with the oracle."""
    for (M, K, B) in ((38016, 2560, 1), (38400, 2560, 2), (19200, 5120, 1), (12800, 6912, 2)):
        z = 0.4219
        W, S = datagen.trits(900 + K + B, M, K, z), datagen.scales(900 + K + B, M, K)
        x, xs = datagen.activations(900 + K + B, B, K)
        rows = np.arange(M)
        acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        ws = bc.make_workspace(M, K)
        st = bc.scales_tile(S, M, K)
        for fmt, Wd, f in (("bitcos", bc.bitcos_pack(W, S).to_device(), bc.bitcos_gemv),
                           ("trit5", bc.plain_to_device(bc.trit5_pack(W), st, M, K), bc.trit5_gemv),
                           ("bit2", bc.plain_to_device(bc.bit2_pack(W), st, M, K), bc.bit2_gemv)):
            for rep in range(2):
                y, acc = f(Wd, xd, xsd, acc_debug=True, workspace=ws)
                torch.cuda.synchronize()
                assert np.array_equal(acc.cpu().numpy()[:, rows], acc_ref), (fmt, M, K, B)
                err = np.abs(y.cpu().numpy().astype(np.float64)[:, rows] - y_ref)
                assert (err <= REL * mag).all(), (fmt, M, K, B)
            assert bc.workspace_status(ws) == 0
            del Wd


def test_multi_launch_two_tiles_per_warp(bc):
    """A multi launch with enough items altogether (eight or more per multiprocessor) runs every
    job with two tiles per decoder warp: jobs of different shapes, among them a small one, one
    whose rows are cut into column blocks and one with a ragged last row block.  Every output
    against the oracle; the same bits from run to run."""
    shapes = [(12800, 2560), (6400, 5120), (64, 2560), (3200, 6912), (1000, 5120), (4097, 2560)]
    for B in (1, 2):
        jobs, refs = [], []
        for i, (M, K) in enumerate(shapes):
            W, S = datagen.trits(1300 + i, M, K, 0.4219), datagen.scales(1300 + i, M, K)
            x, xs = datagen.activations(1300 + i + B, B, K)
            rows = np.arange(M)
            refs.append((rows,) + tuple(oracle.gemv_dense(W, S, x, xs)))
            y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
            jobs.append((bc.bitcos_pack(W, S).to_device(), dev(x), dev(xs), y, bc.make_workspace(M, K)))
        for rep in range(2):
            for j in jobs:
                j[3].fill_(float("nan"))
            bc.bitcos_gemv_multi(jobs)
            torch.cuda.synchronize()
            for (Wd, _, _, y, ws), (rows, acc_ref, y_ref, mag) in zip(jobs, refs):
                yh = y.cpu().numpy().astype(np.float64)
                assert np.isfinite(yh).all(), (Wd.M, Wd.K, B)
                assert (np.abs(yh[:, rows] - y_ref) <= REL * mag).all(), (Wd.M, Wd.K, B)
                assert bc.workspace_status(ws) == 0
        # run to run the same bits (the order of the additions is fixed)
        first = [j[3].clone() for j in jobs]
        bc.bitcos_gemv_multi(jobs)
        torch.cuda.synchronize()
        for j, y0 in zip(jobs, first):
            assert torch.equal(j[3], y0)


def test_multi_host_buffer_entry_point(bc):
    """Several products from host buffers in one call: same results as the device entry point."""
    B = 2
    jobs, refs = [], []
    for i, (M, K) in enumerate([(640, 2560), (96, 6912), (2560, 2560)]):
        W, S = datagen.trits(800 + i, M, K, 0.4219), datagen.scales(800 + i, M, K)
        x, xs = datagen.activations(800 + i, B, K)
        refs.append(oracle.gemv_dense(W, S, x, xs))
        staging = torch.empty(bc.bitcos_gemv_host_staging_bytes(M, K, B), dtype=torch.uint8, device="cuda")
        xh, xsh = torch.from_numpy(x).pin_memory(), torch.from_numpy(xs).pin_memory()
        yh = torch.full((B, M), float("nan"), dtype=torch.float32).pin_memory()
        jobs.append((bc.bitcos_pack(W, S).to_device(), xh.numpy(), xsh.numpy(), yh.numpy(), staging, bc.make_workspace(M, K),
                     (xh, xsh, yh)))
    bc.bitcos_gemv_multi_host([j[:6] for j in jobs])
    for (Wd, xh, xsh, yh, st, ws, _), (acc_ref, y_ref, mag) in zip(jobs, refs):
        err = np.abs(yh.astype(np.float64) - y_ref)
        assert (err <= REL * mag).all()
        y_dev, _ = bc.bitcos_gemv(Wd, dev(xh), dev(xsh), workspace=ws)
        torch.cuda.synchronize()
        assert np.array_equal(y_dev.cpu().numpy(), yh)


def test_layer_shapes_every_output(bc):
    """The largest layer shapes of the benchmark configurations, in the launch configuration
    the benchmark times; every accumulator and every output against the oracle."""
    for (M, K, z, B) in ((6912, 2560, 0.4219, 1), (2560, 6912, 0.4219, 1), (5120, 25600, 0.4711, 2),
                         (8192, 5120, 0.4711, 16), (6912, 2560, 0.4219, 8)):
        W, S = datagen.trits(500 + M, M, K, z), datagen.scales(500 + M, M, K)
        x, xs = datagen.activations(500 + M, B, K)
        rows = np.arange(M)
        acc_ref, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        ws = bc.make_workspace(M, K)
        st = bc.scales_tile(S, M, K)
        for fmt, Wd, f in (("bitcos", bc.bitcos_pack(W, S).to_device(), bc.bitcos_gemv),
                           ("trit5", bc.plain_to_device(bc.trit5_pack(W), st, M, K), bc.trit5_gemv),
                           ("bit2", bc.plain_to_device(bc.bit2_pack(W), st, M, K), bc.bit2_gemv)):
            y, acc = f(Wd, xd, xsd, acc_debug=True, workspace=ws)
            torch.cuda.synchronize()
            assert np.array_equal(acc.cpu().numpy()[:, rows], acc_ref), fmt
            err = np.abs(y.cpu().numpy().astype(np.float64)[:, rows] - y_ref)
            assert (err <= REL * mag).all(), fmt
