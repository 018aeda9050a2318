"""GPU parity at the literal sizes of the benchmark configurations: every int32 group accumulator
bit-exact and every fp32 output within 1e-5 of sum|terms| of the CPU oracle, in the launch
configuration the benchmark times.

  config 1  BitNet-b1.58-2B layer, seven products, one token, all three formats, single and
            fused (multi) launches
  config 2  4096 x 12288 and 12288 x 4096 at five zero densities, one token, all three formats
  config 3  Qwen3-32B-shaped layer (five distinct shapes), 1 / 2 / 4 / 8 / 16 tokens, all three formats
  config 4  128 experts, eight distinct experts per token, 1 / 2 / 4 / 8 / 16 tokens, gate/up and down

Every matrix is generated and packed once per module and reused across formats and batches.
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


def compare(y, acc, acc_ref, y_ref, mag, what):
    torch.cuda.synchronize()
    if acc is not None:
        assert np.array_equal(acc.cpu().numpy(), acc_ref), f"{what}: int32 accumulators differ"
    yv = y.cpu().numpy().astype(np.float64)
    err = np.abs(yv - y_ref)
    assert (err <= REL * mag).all(), f"{what}: worst {np.max(err / np.maximum(mag, 1e-300)):.3e}"
    assert (yv[mag == 0] == 0).all(), what


def three_formats(bc, W, S):
    M, K = W.shape
    st = bc.scales_tile(S, M, K)
    return (("bitcos", bc.bitcos_pack(W, S).to_device(), bc.bitcos_gemv),
            ("trit5", bc.plain_to_device(bc.trit5_pack(W), st, M, K), bc.trit5_gemv),
            ("bit2", bc.plain_to_device(bc.bit2_pack(W), st, M, K), bc.bit2_gemv))


def test_config1_bitnet_layer(bc):
    cfg = datagen.CONFIG_BITNET_2B
    jobs, refs = [], []
    for i, (name, M, K) in enumerate(cfg["shapes"]):
        s = datagen.config_seed(1, i)
        W, S = datagen.trits(s, M, K, cfg["z"]), datagen.scales(s, M, K)
        x, xs = datagen.activations(s, 1, K)
        ref = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        ws = bc.make_workspace(M, K)
        for fmt, Wd, f in three_formats(bc, W, S):
            y, acc = f(Wd, xd, xsd, acc_debug=True, workspace=ws)
            compare(y, acc, *ref, f"config 1 {name} {fmt}")
            if fmt == "bitcos":
                jobs.append((Wd, xd, xsd, torch.full((1, M), float("nan"), dtype=torch.float32, device="cuda"), ws))
                refs.append(ref)
    # the launches the benchmark's step makes: q + k + v, o, gate + up, down
    for group in ((0, 1, 2), (3,), (4, 5), (6,)):
        bc.bitcos_gemv_multi([jobs[i] for i in group])
    for i, (name, M, K) in enumerate(cfg["shapes"]):
        compare(jobs[i][3], None, *refs[i], f"config 1 {name} fused launch")
        assert bc.workspace_status(jobs[i][4]) == 0


@pytest.mark.parametrize("shape", datagen.CONFIG_SWEEP["shapes"], ids=lambda s: s[0])
def test_config2_density_sweep(bc, shape):
    name, M, K = shape
    for zi, z in enumerate(datagen.CONFIG_SWEEP["zs"]):
        s = datagen.config_seed(2, 10 * zi + (0 if name == "wide" else 1))
        W, S = datagen.trits(s, M, K, z), datagen.scales(s, M, K)
        x, xs = datagen.activations(s, 1, K)
        ref = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        ws = bc.make_workspace(M, K)
        for fmt, Wd, f in three_formats(bc, W, S):
            y, acc = f(Wd, xd, xsd, acc_debug=True, workspace=ws)
            compare(y, acc, *ref, f"config 2 {name} z={z} {fmt}")
        assert bc.workspace_status(ws) == 0


QWEN_DISTINCT = [s for s in datagen.CONFIG_QWEN3_32B["shapes"] if s[0] in ("q", "k", "o", "gate", "down")]


@pytest.mark.parametrize("shape", QWEN_DISTINCT, ids=lambda s: s[0])
def test_config3_qwen_layer(bc, shape):
    cfg = datagen.CONFIG_QWEN3_32B
    name, M, K = shape
    i = [s[0] for s in cfg["shapes"]].index(name)
    s = datagen.config_seed(3, i)
    W, S = datagen.trits(s, M, K, cfg["z"]), datagen.scales(s, M, K)
    fmts = three_formats(bc, W, S)
    ws = bc.make_workspace(M, K)
    for B in cfg["batches"]:
        x, xs = datagen.activations(s + 100 * B, B, K)
        ref = oracle.gemv_dense(W, S, x, xs)
        xd, xsd = dev(x), dev(xs)
        for fmt, Wd, f in fmts:
            y, acc = f(Wd, xd, xsd, acc_debug=True, workspace=ws)
            compare(y, acc, *ref, f"config 3 {name} B={B} {fmt}")
            del y, acc
    assert bc.workspace_status(ws) == 0


@pytest.mark.parametrize("proj", ["gate", "down"])
def test_config4_moe_experts(bc, proj):
    cfg = datagen.CONFIG_QWEN3_MOE
    E, top_k, z = cfg["n_experts"], cfg["top_k"], cfg["z"]
    M, K = (768, 2048) if proj == "gate" else (2048, 768)
    base = datagen.config_seed(4, 0 if proj == "gate" else 500)
    Ws = [datagen.trits(base + e, M, K, z) for e in range(E)]
    Ss = [datagen.scales(base + e, M, K) for e in range(E)]
    sts = [bc.scales_tile(Ss[e], M, K) for e in range(E)]
    formats = (("bitcos", bc.DeviceExperts([bc.bitcos_pack(Ws[e], Ss[e]).to_device() for e in range(E)]), bc.bitcos_gemv_grouped),
               ("trit5", bc.DeviceExperts([bc.plain_to_device(bc.trit5_pack(Ws[e]), sts[e], M, K) for e in range(E)]), bc.trit5_gemv_grouped),
               ("bit2", bc.DeviceExperts([bc.plain_to_device(bc.bit2_pack(Ws[e]), sts[e], M, K) for e in range(E)]), bc.bit2_gemv_grouped))
    for tokens in cfg["batches"]:
        ids = datagen.expert_choices(base + tokens, tokens, E, top_k)
        pair_expert = ids.reshape(-1)
        if proj == "gate":
            # gate / up: every pair of a token reads that token's activations
            x, xs = datagen.activations(base + 7 * tokens, tokens, K)
            pair_xrow = np.repeat(np.arange(tokens, dtype=np.int32), top_k)
        else:
            # down: every (token, expert) pair has its own input row
            x, xs = datagen.activations(base + 7 * tokens, tokens * top_k, K)
            pair_xrow = np.arange(tokens * top_k, dtype=np.int32)
        order, ge, gb, xr, mx = bc.group_pairs(pair_expert, pair_xrow)
        acc_ref, y_ref, mag = oracle.grouped_dense(Ws, Ss, pair_expert[order], pair_xrow[order], x, xs)
        ws = bc.make_workspace(M, K, copies=len(ge))
        for fmt, experts, f in formats:
            for rep in range(2):
                y, acc = f(experts, dev(ge), dev(gb), dev(xr), mx, dev(x), dev(xs), acc_debug=True, workspace=ws)
                compare(y, acc, acc_ref, y_ref, mag, f"config 4 {proj} tokens={tokens} {fmt} rep{rep}")
            assert bc.workspace_status(ws) == 0
