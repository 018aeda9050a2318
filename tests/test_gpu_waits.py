"""The give-up path of the bounded waits, exercised without faulting anything: a wait that can never
be satisfied runs out after its limit, the status word reads 1, the kernel returns normally, and the
library keeps working -- on a fresh workspace and on the marked one once it is cleared."""
import numpy as np
import pytest

import datagen
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bc():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_16338_b200 as m
    from paper_2609_16338_b200 import build
    build.build()
    m.load_library()
    return m


def test_a_wait_that_runs_out_sets_the_status_word_and_returns(bc):
    M, K = 320, 2560
    W, S = datagen.trits(31, M, K, 0.42), datagen.scales(31, M, K)
    x, xs = datagen.activations(31, 1, K)
    _, y_ref, mag = oracle.gemv_dense(W, S, x, xs)
    Wd = bc.bitcos_pack(W, S).to_device()
    xd, xsd = torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda()

    ws = bc.make_workspace(M, K)
    assert bc.workspace_status(ws) == 0
    waited = bc.bitcos_wait_probe(ws, limit_ns=1_000_000)          # one millisecond
    assert bc.workspace_status(ws) == 1
    assert 1_000_000 <= waited < 50_000_000                        # it polled for the limit, not for ever
    # the context is intact: an ordinary product on a fresh workspace is right ...
    y, _ = bc.bitcos_gemv(Wd, xd, xsd, workspace=bc.make_workspace(M, K))
    torch.cuda.synchronize()
    assert (np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= 1e-5 * mag).all()
    # ... and so is one on the marked workspace once it has been cleared again
    ws.zero_()
    y2, _ = bc.bitcos_gemv(Wd, xd, xsd, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(y, y2) and bc.workspace_status(ws) == 0


def test_status_of_the_built_in_scratch_array(bc):
    M, K = 96, 6912
    W, S = datagen.trits(32, M, K, 0.42), datagen.scales(32, M, K)
    x, xs = datagen.activations(32, 1, K)
    Wd = bc.bitcos_pack(W, S).to_device()
    y = torch.empty((1, M), dtype=torch.float32, device="cuda")
    bc.bitcos_gemv_static(Wd, torch.from_numpy(x).cuda(), torch.from_numpy(xs).cuda(), y)
    assert bc.bitcos_gemv_static_status() == 0
