"""GPU parity of the coarse-to-fine proxy (Section 4.1) against the oracle's literal sort-and-diff."""
import math

import numpy as np
import pytest
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs

pytestmark = pytest.mark.gpu


def _run(mats, K=4, tau_c=1.5, tau_f=50.0):
    dev = [torch.from_numpy(np.ascontiguousarray(m)).cuda() for m in mats]
    ws = torch.empty(B.rwkvq_proxy_workspace_bytes(len(dev)), dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)  # contents on entry must not matter
    return B.rwkvq_proxy_select(dev, K, tau_c, tau_f, ws)


def _close(a, b, rel=1e-9):
    return abs(a - b) <= rel * max(1.0, abs(b))


@pytest.mark.parametrize("K", [2, 4, 6, 8])
def test_proxy_matches_oracle(K):
    mats = [inputs.gen_weight(0, 512, 512, "gauss"), inputs.gen_weight(1, 256, 768, "student"),
            inputs.gen_weight(2, 128, 384, "uniform"), inputs.gen_weight(3, 3, 37, "gauss"),
            (np.arange(4096).reshape(64, 64) % 17 - 8).astype(np.float16)]
    big = inputs.gen_weight(4, 64, 64, "gauss").copy()
    big[0, 0], big[5, 7] = np.float16(900.0), np.float16(-40000.0)   # outside the shared-memory window
    mats.append(big)
    pc, pf, phi = _run(mats, K=K)
    for m, a, b, p in zip(mats, pc, pf, phi):
        ra, rb = orc.proxy(m.astype(np.float64), K=K)
        assert _close(a, ra) and _close(b, rb, 1e-8), (a, ra, b, rb)
        assert p == orc.select(ra, rb, 1.5, 50.0)


def test_proxy_full_size_matrix_and_threshold_between_clusters():
    g = inputs.gen_weight(10, 2048, 2048, "gauss")
    t = inputs.gen_weight(11, 2048, 2048, "student")
    pc, pf, _ = _run([g, t])
    rg, rt = orc.proxy(g.astype(np.float64)), orc.proxy(t.astype(np.float64))
    assert _close(pc[0], rg[0]) and _close(pc[1], rt[0]) and _close(pf[0], rg[1], 1e-8) and _close(pf[1], rt[1], 1e-8)
    assert pc[0] < pc[1]
    tau = 0.5 * (pc[0] + pc[1])
    _, _, phi = _run([g, t], tau_c=tau, tau_f=math.inf)
    assert list(phi) == [B.RWKVQ_SQ, B.RWKVQ_VQ]


def test_proxy_degenerate_and_nonfinite():
    const = np.full((16, 16), 0.25, np.float16)
    zeros = np.zeros((8, 8), np.float16)
    zeros[0, 0] = np.float16(-0.0)
    pc, pf, phi = _run([const, zeros])
    assert math.isinf(pc[0]) and math.isinf(pf[0]) and math.isinf(pc[1]) and list(phi) == [0, 0]
    bad = inputs.gen_weight(0, 16, 16).copy()
    bad[3, 3] = np.float16(np.nan)
    with pytest.raises(B.RwkvqError) as e:
        _run([bad])
    assert e.value.status == 4
    with pytest.raises(B.RwkvqError):
        _run([const], K=9)


def test_proxy_family_matches_oracle():
    # Section 5.3's other statistics of G', from the same histogram pass
    mats = [inputs.gen_weight(0, 512, 512, "gauss"), inputs.gen_weight(1, 256, 768, "student"),
            inputs.gen_weight(2, 128, 384, "uniform"), inputs.gen_weight(3, 3, 37, "gauss"),
            (np.arange(4096).reshape(64, 64) % 17 - 8).astype(np.float16),
            (np.arange(2048).reshape(32, 64) * 0.25 - 100.0).astype(np.float16),      # no ties: minimum gap > 0
            np.full((16, 16), 0.25, np.float16)]
    dev = [torch.from_numpy(np.ascontiguousarray(m)).cuda() for m in mats]
    ws = torch.empty(B.rwkvq_proxy_workspace_bytes(len(dev)), dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)
    got = B.rwkvq_proxy_family(dev, ws)
    for i, m in enumerate(mats):
        ref = orc.proxy_family(m.astype(np.float64))
        for k, v in ref.items():
            if math.isinf(v):
                assert math.isinf(got[k][i]), (i, k)
            else:
                assert abs(got[k][i] - v) <= 1e-9 * abs(v) + 1e-13, (i, k, got[k][i], v)   # equal gaps: exact 0 vs rounding
    # the entropy is the coarse proxy in other words
    pc, _, _ = _run(mats[:6], K=2)
    for i in range(6):
        assert _close(math.log(mats[i].size - 1) - got["ie"][i], pc[i])


def test_thresholds_for_a_target_sq_share():
    # Section 5.1: thresholds set so that a stated share of the matrices uses SQ
    mats = [inputs.gen_weight(20 + i, 128, 256, "student" if i % 5 == 0 else "gauss") for i in range(10)]
    pc, _, _ = _run(mats, tau_c=math.inf, tau_f=math.inf)
    tau = B.rwkvq_tau_for_fraction(pc, 0.8)
    assert tau == orc.tau_for_fraction(pc, 0.8)
    _, _, phi = _run(mats, tau_c=tau, tau_f=math.inf)
    assert int(phi.sum()) == 8 and phi[0] == B.RWKVQ_VQ and phi[5] == B.RWKVQ_VQ


def _typed(a32, dtype):
    """float32 array -> (float64 values as the device will see them, CUDA tensor of `dtype`)."""
    t = torch.from_numpy(np.ascontiguousarray(a32, dtype=np.float32)).cuda().to(dtype)
    return t.double().cpu().numpy(), t


def _close_arr(a, b, rel):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    inf = np.isinf(b)
    assert np.array_equal(np.isinf(a), inf)
    assert (np.abs(a[~inf] - b[~inf]) <= rel * np.maximum(1.0, np.abs(b[~inf]))).all(), float(np.abs(a[~inf] - b[~inf]).max())


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape,seg", [((40, 300), (1, 300)), ((40, 300), (16, 128)), ((512, 512), (256, 256)),
                                       ((33, 70), (8, 64)), ((3, 5000), (1, 5000))])
def test_proxy_segments_match_oracle_per_tile(dtype, shape, seg):
    if dtype == torch.float32 and seg[0] * seg[1] > 32768:
        seg = (seg[0] // 2, seg[1])             # an fp32 tile holds half as many elements
    rng = np.random.default_rng(shape[0] * 7 + seg[1])
    a = rng.standard_normal(shape).astype(np.float32) * 0.02
    a[::5, ::3] = np.float32(0.0078125)          # ties across tiles
    a[0, : min(shape[1], seg[1])] = np.float32(0.25) if seg[0] == 1 else a[0, : min(shape[1], seg[1])]   # a constant channel
    vals, dev = _typed(a, dtype)
    pc, pf, phi = B.rwkvq_proxy_segments(dev, seg[0], seg[1], 4, 3.0, 1e30)
    rpc, rpf = orc.proxy_segments(vals, min(seg[0], shape[0]), min(seg[1], shape[1]), K=4)
    _close_arr(pc, rpc, 1e-9)
    _close_arr(pf, rpf, 1e-8)
    want = np.array([[orc.select(x, y, 3.0, 1e30) for x, y in zip(r1, r2)] for r1, r2 in zip(rpc, rpf)])
    far = np.abs(rpc - 3.0) > 1e-6           # a tile whose P_c sits on the threshold may fall either way
    assert np.array_equal(phi[far], want[far])
    if seg[0] == 1:
        assert np.isinf(pc[0, 0]) and phi[0, 0] == B.RWKVQ_VQ


def test_proxy_segments_k_and_one_element_tiles():
    a = np.arange(35, dtype=np.float32).reshape(5, 7) ** 2
    vals, dev = _typed(a, torch.float32)
    for K in (2, 8):
        pc, pf, _ = B.rwkvq_proxy_segments(dev, 2, 3, K, 1.0, 1.0)
        rpc, rpf = orc.proxy_segments(vals, 2, 3, K=K)
        _close_arr(pc, rpc, 1e-9)
        _close_arr(pf, rpf, 1e-8)
    assert np.isinf(pc[2, 2])                # the corner tile holds one element


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_proxy_whole_matrix_other_types_match_oracle(dtype):
    rng = np.random.default_rng(17)
    for (oc, ic, kind) in ((700, 900, "gauss"), (256, 1024, "student"), (64, 64, "ties")):
        if kind == "gauss":
            a = rng.standard_normal((oc, ic)).astype(np.float32) * 0.02
        elif kind == "student":
            a = rng.standard_t(3.0, (oc, ic)).astype(np.float32) * 0.01
        else:
            a = rng.integers(-3, 4, (oc, ic)).astype(np.float32) * 0.5
        vals, dev = _typed(a, dtype)
        pc, pf, phi = B.rwkvq_proxy_select_typed(dev, 4, 1e30, 1e30)
        rpc, rpf = orc.proxy(vals, K=4)
        assert abs(pc - rpc) <= 1e-9 * max(1.0, abs(rpc)), (kind, pc, rpc)
        assert abs(pf - rpf) <= 1e-8 * max(1.0, abs(rpf)), (kind, pf, rpf)
        assert phi == B.RWKVQ_SQ
    # the fp16 route through the same wrapper agrees with the batched call
    vals, dev = _typed(rng.standard_normal((128, 256)).astype(np.float32) * 0.02, torch.float16)
    pc, pf, _ = B.rwkvq_proxy_select_typed(dev, 4, 1e30, 1e30)
    rpc, rpf = orc.proxy(vals, K=4)
    assert abs(pc - rpc) <= 1e-9 * max(1.0, abs(rpc)) and abs(pf - rpf) <= 1e-8 * max(1.0, abs(rpf))


def test_proxy_segments_and_typed_errors():
    z = torch.zeros((300, 300), dtype=torch.float32, device="cuda")
    with pytest.raises(B.RwkvqError):
        B.rwkvq_proxy_segments(z, 300, 300, 4, 1.0, 1.0)            # 90 000 fp32 elements in one tile
    h = torch.zeros((300, 300), dtype=torch.float16, device="cuda")
    with pytest.raises(B.RwkvqError):
        B.rwkvq_proxy_segments(h, 300, 300, 4, 1.0, 1.0)            # 90 000 > 65 536
    pc, pf, phi = B.rwkvq_proxy_segments(h, 100, 300, 4, 1.0, 1.0)   # constant tiles
    assert np.isinf(pc).all() and (phi == B.RWKVQ_VQ).all()
    for dt in (torch.float16, torch.bfloat16, torch.float32):
        bad = torch.ones((8, 64), dtype=dt, device="cuda")
        bad[3, 5] = float("nan")
        with pytest.raises(B.RwkvqError):
            B.rwkvq_proxy_segments(bad, 4, 64, 4, 1.0, 1.0)
        if dt != torch.float16:
            with pytest.raises(B.RwkvqError):
                B.rwkvq_proxy_select_typed(bad, 4, 1.0, 1.0)
    with pytest.raises(B.RwkvqError):
        B.rwkvq_proxy_segments(h, 16, 16, 9, 1.0, 1.0)              # K out of range
