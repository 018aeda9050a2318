"""The phased launch (bitcos_gemv_phased): jobs in dependency order inside one launch.  Against the
oracle, bit for bit against one bitcos_gemv_multi call per phase, and with a real dependency: a job
whose activations ARE the bytes another job of the phase before writes."""
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
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def make_jobs(bc, shapes, B, seed, z=0.4219):
    jobs, refs = [], []
    for i, (M, K) in enumerate(shapes):
        W, S = datagen.trits(seed + i, M, K, z), datagen.scales(seed + i, M, K)
        x, xs = datagen.activations(seed + i, B, K)
        refs.append(oracle.gemv_dense(W, S, x, xs))
        y = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
        jobs.append((bc.bitcos_pack(W, S).to_device(), dev(x), dev(xs), y, bc.make_workspace(M, K)))
    return jobs, refs


LAYER = [(2560, 2560), (640, 2560), (640, 2560), (2560, 2560), (6912, 2560), (6912, 2560), (2560, 6912)]
LAYER_PHASES = [0, 0, 0, 1, 2, 2, 3]


@pytest.mark.parametrize("B", [1, 2])
def test_decoder_layer_in_one_launch(bc, B):
    jobs, refs = make_jobs(bc, LAYER, B, 4000 + B)
    sync = bc.make_phased_sync()
    for rep in range(3):                      # the sync words and the workspaces must come back clean
        for j in jobs:
            j[3].fill_(float("nan"))
        bc.bitcos_gemv_phased(jobs, LAYER_PHASES, sync)
        torch.cuda.synchronize()
        for (Wd, _, _, y, ws), (acc_ref, y_ref, mag) in zip(jobs, refs):
            err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
            assert (err <= REL * mag).all(), (rep, Wd.M, Wd.K)
            assert bc.workspace_status(ws) == 0
        assert int(sync.view(torch.int32).abs().sum()) == 0
    phased = [j[3].clone() for j in jobs]
    for group in ((0, 1, 2), (3,), (4, 5), (6,)):
        bc.bitcos_gemv_multi([jobs[i] for i in group])
    torch.cuda.synchronize()
    for j, y0 in zip(jobs, phased):
        assert torch.equal(j[3], y0)


def test_odd_shapes_and_phase_layouts(bc):
    """Ragged row counts, rows cut into column blocks, a phase with one tiny job, two phases only,
    a single phase, and all four phases with one job each."""
    shapes = [(100, 384), (33, 6912), (1000, 512), (64, 128), (320, 1280), (96, 2560)]
    jobs, refs = make_jobs(bc, shapes, 1, 4100, z=0.35)
    for phases in ([0, 0, 0, 1, 1, 1], [0, 0, 0, 0, 0, 0], [0, 1, 2, 3, 3, 3], [0, 1, 1, 1, 2, 3]):
        sync = bc.make_phased_sync()
        for rep in range(2):
            for j in jobs:
                j[3].fill_(float("nan"))
            bc.bitcos_gemv_phased(jobs, phases, sync)
            torch.cuda.synchronize()
            for (Wd, _, _, y, ws), (acc_ref, y_ref, mag) in zip(jobs, refs):
                err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
                assert (err <= REL * mag).all(), (phases, Wd.M, Wd.K)
                assert bc.workspace_status(ws) == 0


def test_a_job_reads_what_the_phase_before_wrote(bc):
    """Phase 1's activations are the raw bytes of phase 0's fp32 outputs (640 floats = 2560 int8), poisoned
    before the launch: the result is right only if phase 1 reads them after phase 0 has written them all."""
    M0, K0, M1 = 640, 2560, 6912
    K1 = 4 * M0
    W0, S0 = datagen.trits(4200, M0, K0, 0.42), datagen.scales(4200, M0, K0)
    W1, S1 = datagen.trits(4201, M1, K1, 0.42), datagen.scales(4201, M1, K1)
    x0, xs0 = datagen.activations(4200, 1, K0)
    xs1 = np.array([0.0123], dtype=np.float32)
    Wd0, Wd1 = bc.bitcos_pack(W0, S0).to_device(), bc.bitcos_pack(W1, S1).to_device()
    y0 = torch.empty((1, M0), dtype=torch.float32, device="cuda")
    y1 = torch.empty((1, M1), dtype=torch.float32, device="cuda")
    x1 = y0.view(torch.int8).view(1, K1)                      # the same memory, seen as int8 activations
    # a second, large job in phase 0 keeps most thread blocks busy while the small one finishes
    Wb, Sb = datagen.trits(4202, 12800, 2560, 0.42), datagen.scales(4202, 12800, 2560)
    xb, xsb = datagen.activations(4202, 1, 2560)
    yb = torch.empty((1, 12800), dtype=torch.float32, device="cuda")
    jobs = [(Wd0, dev(x0), dev(xs0), y0, bc.make_workspace(M0, K0)),
            (bc.bitcos_pack(Wb, Sb).to_device(), dev(xb), dev(xsb), yb, bc.make_workspace(12800, 2560)),
            (Wd1, x1, dev(xs1), y1, bc.make_workspace(M1, K1))]
    sync = bc.make_phased_sync()
    for rep in range(3):
        y0.fill_(float("nan"))
        y1.fill_(float("nan"))
        bc.bitcos_gemv_phased(jobs, [0, 0, 1], sync)
        torch.cuda.synchronize()
        _, y0_ref, mag0 = oracle.gemv_dense(W0, S0, x0, xs0)
        assert (np.abs(y0.cpu().numpy().astype(np.float64) - y0_ref) <= REL * mag0).all()
        x1_host = y0.cpu().numpy().view(np.int8).reshape(1, K1)
        acc1, y1_ref, mag1 = oracle.gemv_dense(W1, S1, x1_host, xs1)
        assert (np.abs(y1.cpu().numpy().astype(np.float64) - y1_ref) <= REL * mag1).all(), rep
        assert all(bc.workspace_status(j[4]) == 0 for j in jobs)


def test_phases_from_host_buffers_in_one_call(bc):
    """One copy in, one launch per phase, one copy out, one wait: same results as the device entry points."""
    B = 2
    mats = []
    for i, (M, K) in enumerate(LAYER):
        W, S = datagen.trits(4300 + i, M, K, 0.4219), datagen.scales(4300 + i, M, K)
        mats.append((W, S, bc.bitcos_pack(W, S).to_device(), bc.make_workspace(M, K)))
    hp = bc.HostPhases([(m[2], m[3]) for m in mats], LAYER_PHASES, batch=B)
    # (the first call enqueues the step directly, the second records it, from the third on it is replayed)
    for rep in range(5):
        refs = []
        for i, (W, S, Wd, ws) in enumerate(mats):
            x, xs = datagen.activations(4300 + 10 * rep + i, B, Wd.K)
            hp.x[i][:] = x
            hp.x_scale[i][:] = xs
            refs.append(oracle.gemv_dense(W, S, x, xs))
        ys = hp.run()
        for i, (acc_ref, y_ref, mag) in enumerate(refs):
            assert (np.abs(ys[i].astype(np.float64) - y_ref) <= REL * mag).all(), (rep, i)
            y_dev, _ = bc.bitcos_gemv(mats[i][2], dev(hp.x[i].copy()), dev(hp.x_scale[i].copy()), workspace=mats[i][3])
            torch.cuda.synchronize()
            assert np.array_equal(y_dev.cpu().numpy(), ys[i])


def test_recorded_host_step_follows_weights_repacked_in_place(bc):
    """A step seen before is replayed as a recorded graph.  The record holds entry offsets taken from the
    host copy of tile_off; when different weights are packed into the SAME buffers (same descriptor, new
    offsets), the next call must notice and still return the new product."""
    B = 1
    shapes = [(640, 2560), (320, 1280)]
    Wh = [datagen.trits(4400 + i, M, K, 0.4219) for i, (M, K) in enumerate(shapes)]
    Sh = [datagen.scales(4400 + i, M, K) for i, (M, K) in enumerate(shapes)]
    packs = [bc.bitcos_pack(W, S) for W, S in zip(Wh, Sh)]
    devs = [p.to_device() for p in packs]
    hp = bc.HostPhases([(d, bc.make_workspace(M, K)) for d, (M, K) in zip(devs, shapes)], [0, 1], batch=B)

    def check(tag):
        for rep in range(4):
            refs = []
            for i, (M, K) in enumerate(shapes):
                x, xs = datagen.activations(4400 + 7 * rep + i, B, K)
                hp.x[i][:] = x
                hp.x_scale[i][:] = xs
                refs.append(oracle.gemv_dense(Wh[i], Sh[i], x, xs))
            ys = hp.run()
            for i, (acc_ref, y_ref, mag) in enumerate(refs):
                assert (np.abs(ys[i].astype(np.float64) - y_ref) <= REL * mag).all(), (tag, rep, i)

    check("first weights")
    # new weights of another density into the same device arrays and the same host copy of the entry offsets
    for i, (M, K) in enumerate(shapes):
        Wh[i] = datagen.trits(4500 + i, M, K, 0.6)
        Sh[i] = datagen.scales(4500 + i, M, K)
        p2 = bc.bitcos_pack(Wh[i], Sh[i])
        d = devs[i]
        assert p2.signs.size <= d.signs.numel()          # fewer nonzero weights than before: the sign vector fits
        off = p2.tile_off_buf if p2.tile_off_buf is not None else p2.tile_off
        d.bitmap.copy_(torch.from_numpy(p2.bitmap.view(np.int32)))
        d.signs[:p2.signs.size].copy_(torch.from_numpy(p2.signs.view(np.int32)))
        d.tile_off[:off.size].copy_(torch.from_numpy(off.view(np.int32)))
        d.scales.copy_(torch.from_numpy(p2.scales.view(np.int16)))
        d.tile_off_host[:] = p2.tile_off
    torch.cuda.synchronize()
    check("weights repacked in place")


def test_host_steps_from_two_threads(bc):
    """bitcos_gemv_phases_host from two host threads at once, each with its own matrices, blocks and stream (the
    records of seen steps are shared between threads, recording happens on one stream of the library's own)."""
    import threading
    B = 1
    shapes = [(640, 2560), (96, 1280)]
    errors = []

    def worker(t):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            Wh = [datagen.trits(4600 + 10 * t + i, M, K, 0.4219) for i, (M, K) in enumerate(shapes)]
            Sh = [datagen.scales(4600 + 10 * t + i, M, K) for i, (M, K) in enumerate(shapes)]
            devs = [bc.bitcos_pack(W, S).to_device() for W, S in zip(Wh, Sh)]
            hp = bc.HostPhases([(d, bc.make_workspace(M, K)) for d, (M, K) in zip(devs, shapes)], [0, 1], batch=B)
            with torch.cuda.stream(stream):
                for rep in range(12):
                    refs = []
                    for i, (M, K) in enumerate(shapes):
                        x, xs = datagen.activations(4600 + 100 * t + 7 * rep + i, B, K)
                        hp.x[i][:] = x
                        hp.x_scale[i][:] = xs
                        refs.append(oracle.gemv_dense(Wh[i], Sh[i], x, xs))
                    ys = hp.run()
                    for i, (acc_ref, y_ref, mag) in enumerate(refs):
                        if not (np.abs(ys[i].astype(np.float64) - y_ref) <= REL * mag).all():
                            errors.append((t, rep, i))
        except Exception as e:          # noqa: BLE001 (reported to the main thread)
            errors.append((t, repr(e)))

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
