"""GPU parity of the prefill product (rwkvq_gemm_prefill: dequantise to bf16 tiles, tcgen05 MMA, fp32
accumulation) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _bf16(a32):
    """float32 array -> (float32 array holding the bf16-rounded values, torch bf16 device tensor)."""
    bits = inputs.to_bf16_bits(a32)
    vals = inputs.bf16_bits_to_f32(bits)
    return vals, torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _run(W, mu, X_dev, xprev0_dev, M, y_dtype=torch.float32):
    Y = torch.full((M, W.oc), float("nan"), dtype=y_dtype, device="cuda")
    nbytes = B.rwkvq_prefill_workspace_bytes(W.desc, M, mu is not None)
    assert nbytes > 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)       # contents on entry must not matter
    B.rwkvq_gemm_prefill(W.desc, W.dev, None if mu is None else mu.desc, None if mu is None else mu.dev,
                         X_dev, xprev0_dev, M, Y, ws)
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 0
    return Y


def _reference(W, mu, Xv, xprev0v):
    X64 = Xv.astype(np.float64)
    if mu is None:
        xm = X64
    else:
        prev = orc.prefill_prev(X64, None if xprev0v is None else xprev0v.astype(np.float64))
        xm = orc.token_shift(X64, prev, mu.w_hat)
    return xm


def _check(W, mu, M, seed, with_prev0=True, y_dtype=torch.float32, sample_tokens=None):
    x = inputs.gen_activation(seed, M, W.ic, n_outliers=8)
    Xv, Xd = _bf16(x)
    p0v, p0d = (None, None)
    if mu is not None and with_prev0:
        p0v, p0d = _bf16(inputs.gen_activation(seed + 1, 1, W.ic, n_outliers=8))
        p0v = p0v.reshape(-1)
        p0d = p0d.reshape(-1)
    Y = _run(W, mu, Xd, p0d, M, y_dtype).float().cpu().numpy().astype(np.float64)
    xm = _reference(W, mu, Xv, p0v)
    rows = np.arange(M) if sample_tokens is None else np.asarray(sample_tokens)
    ref = orc.gemv(W.w_hat, xm[rows])
    tol = orc.tolerance(W.w_hat, xm[rows])
    if y_dtype == torch.bfloat16:
        tol = tol + np.abs(ref) * 2.0 ** -8
    err = np.abs(Y[rows] - ref)
    assert np.isfinite(Y).all()
    ratio = float((err / np.maximum(tol, 1e-300)).max())
    assert (err <= tol).all(), f"max err/tol = {ratio}"
    return ratio


@pytest.mark.parametrize("fmt", ["sq", "vq6", "vq8"])
@pytest.mark.parametrize("M", [1, 77, 256, 300])
def test_prefill_small_matches_oracle(fmt, M):
    oc, ic = 256, 512
    W = (H.pack_sq(H.random_sq_codes(M + 3, oc, ic)) if fmt == "sq"
         else H.pack_vq(H.random_vq_codes(M + 5, oc, ic, 6 if fmt == "vq6" else 8), 6 if fmt == "vq6" else 8))
    mu = H.pack_mu(H.random_mu_codes(M + 7, ic))
    _check(W, mu, M, seed=M)
    _check(W, None, M, seed=M + 1)
    _check(W, mu, M, seed=M + 2, with_prev0=False)


def test_prefill_identity_probe_returns_bf16_rounded_decoded_weights():
    # X = I (bf16 ones are exact), no mix: Y[t][i] = bf16_rne(w_hat[i][t]) exactly (adding zeros is exact)
    for W in (H.pack_sq(H.random_sq_codes(11, 384, 512)), H.pack_vq(H.random_vq_codes(12, 256, 512, 6), 6),
              H.pack_vq(H.random_vq_codes(13, 256, 512, 8), 8)):
        M = W.ic
        eye = np.eye(M, dtype=np.float32)
        _, Xd = _bf16(eye)
        Y = _run(W, None, Xd, None, M).cpu().numpy()
        assert np.array_equal(Y, orc.bf16_rne(W.w_hat).T)


def test_prefill_odd_shapes_and_bf16_output():
    W = H.pack_sq(H.random_sq_codes(21, 48, 384))        # rows and columns padded inside the image
    _check(W, H.pack_mu(H.random_mu_codes(22, 384)), 130, seed=23)
    W = H.pack_sq(H.random_sq_codes(24, 256, 1024))
    _check(W, None, 513, seed=25, y_dtype=torch.bfloat16)


@pytest.mark.parametrize("fmt", ["sq", "vq6"])
def test_prefill_7b_shape_sampled(fmt):
    oc, ic, M = 4096, 4096, 2048
    W = H.pack_sq(H.random_sq_codes(31, oc, ic)) if fmt == "sq" else H.pack_vq(H.random_vq_codes(32, oc, ic, 6), 6)
    mu = H.pack_mu(H.random_mu_codes(33, ic))
    toks = [0, 1, 255, 256, 257, 1023, 1024, 2046, 2047]
    _check(W, mu, M, seed=34, sample_tokens=toks)


# The kernel is persistent: with more output tiles (256 weight rows x 256 tokens) than SMs a CTA works
# through several tiles, carrying the phases of its barriers and handing the accumulators back and
# forth between the tensor-core issue thread and the epilogue warps.  Every case below has more than
# 148 tiles; (oc = 640: five chunks, so the last row pair has no second half).
@pytest.mark.parametrize("fmt,oc,ic,M", [
    ("sq", 14336, 512, 2048),      # 56 row pairs x 8 token tiles = 448 tiles, short K
    ("vq6", 7168, 256, 3000),      # 28 x 12 = 336 tiles, ragged last token tile
    ("vq8", 2048, 512, 5120),      # 8 x 20 = 160 tiles
    ("sq", 640, 256, 12800),       # 3 x 50 = 150 tiles, second half of the last row pair absent
    ("vq6", 1280, 512, 8192),      # 5 x 32 = 160 tiles
])
def test_prefill_several_tiles_per_cta(fmt, oc, ic, M):
    bits = 6 if fmt == "vq6" else 8
    W = H.pack_sq(H.random_sq_codes(oc + M, oc, ic)) if fmt == "sq" else H.pack_vq(H.random_vq_codes(oc + M, oc, ic, bits), bits)
    mu = H.pack_mu(H.random_mu_codes(oc + 1, ic))
    rng = np.random.default_rng(M)
    toks = sorted(set([0, 1, 255, 256, 257, M // 2, M - 257, M - 256, M - 2, M - 1]) | set(int(t) for t in rng.integers(0, M, 40)))
    _check(W, mu, M, seed=oc + ic, sample_tokens=toks)


def test_prefill_identity_probe_over_several_tiles_per_cta():
    # X = [I; I; ...] stacked to M tokens: every block of ic tokens returns bf16_rne(w_hat) transposed,
    # bit for bit, whichever tile of whichever CTA computed it (the zeros added in the tensor core are exact)
    oc, ic, reps = 5120, 256, 8                      # 20 row pairs x 8 token tiles = 160 tiles
    W = H.pack_sq(H.random_sq_codes(5, oc, ic))
    M = ic * reps
    _, Xd = _bf16(np.tile(np.eye(ic, dtype=np.float32), (reps, 1)))
    Y = _run(W, None, Xd, None, M).cpu().numpy()
    expect = orc.bf16_rne(W.w_hat).T
    for r in range(reps):
        assert np.array_equal(Y[r * ic:(r + 1) * ic], expect), f"block {r}"


@pytest.mark.parametrize("fmt,oc,ic", [("sq", 14336, 4096), ("sq", 4096, 14336), ("vq6", 14336, 4096), ("vq6", 4096, 14336)])
def test_prefill_channel_mix_shapes_of_the_7b_layer_sampled(fmt, oc, ic):
    # the two 14336-wide products of the timed prefill layer at M = 2048 (448 and 128 tiles), on sampled tokens
    M = 2048
    W = H.pack_sq(H.random_sq_codes(61, oc, ic)) if fmt == "sq" else H.pack_vq(H.random_vq_codes(62, oc, ic, 6), 6)
    mu = H.pack_mu(H.random_mu_codes(63, ic)) if oc > ic else None     # the channel-mix key takes the token shift
    toks = [0, 1, 255, 256, 511, 512, 1023, 1024, 1500, 2046, 2047]
    _check(W, mu, M, seed=64, sample_tokens=toks)


def test_prefill_argument_errors():
    W = H.pack_sq(H.random_sq_codes(41, 128, 256))
    X = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((4, 128), dtype=torch.float32, device="cuda")
    ws = torch.zeros(B.rwkvq_prefill_workspace_bytes(W.desc, 4, False), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemm_prefill(W.desc, W.dev, None, None, X, None, 4, Y, ws[:1024])
    assert e.value.status == 5
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemm_prefill(W.desc, W.dev, None, None, X, None, 0, Y, ws)
    assert e.value.status == 1
    mu = H.pack_mu(H.random_mu_codes(42, 512))
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemm_prefill(W.desc, W.dev, mu.desc, mu.dev, X, None, 4, Y, ws)
    assert e.value.status == 2


def test_prefill_grouped_products_of_mixed_formats_and_lengths():
    """One persistent launch over five products that differ in format, contraction length, row count and
    token-shift use: every output equals the oracle's, and the single-product call gives the same bits."""
    M = 300
    specs = [("sq", 384, 1024, True), ("vq6", 256, 512, True), ("vq8", 512, 768, False), ("sq", 48, 384, True),
             ("sq", 640, 2048, False)]
    prods, entries = [], []
    for i, (fmt, oc, ic, has_mu) in enumerate(specs):
        W = (H.pack_sq(H.random_sq_codes(400 + i, oc, ic)) if fmt == "sq"
             else H.pack_vq(H.random_vq_codes(410 + i, oc, ic, 6 if fmt == "vq6" else 8), 6 if fmt == "vq6" else 8))
        mu = H.pack_mu(H.random_mu_codes(420 + i, ic)) if has_mu else None
        Xv, Xd = _bf16(inputs.gen_activation(430 + i, M, ic, n_outliers=8))
        p0v, p0d = (None, None)
        if has_mu and i % 2 == 0:
            p0v, p0d = _bf16(inputs.gen_activation(440 + i, 1, ic, n_outliers=8))
            p0v, p0d = p0v.reshape(-1), p0d.reshape(-1)
        Y = torch.full((M, oc), float("nan"), dtype=torch.float32, device="cuda")
        ws = torch.empty(B.rwkvq_prefill_workspace_bytes(W.desc, M, has_mu), dtype=torch.uint8, device="cuda")
        ws.fill_(0xCD)
        prods.append((W, mu, Xv, Xd, p0v, p0d, Y))
        entries.append(dict(desc=W.desc, W=W.dev, mu_desc=None if mu is None else mu.desc, mu=None if mu is None else mu.dev,
                            X=Xd, xprev0=p0d, Y=Y, workspace=ws))
    for _ in range(2):      # the scheduling word is cleared by every call
        B.rwkvq_gemm_prefill_grouped(entries, M)
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 0
    for (W, mu, Xv, Xd, p0v, p0d, Y) in prods:
        xm = _reference(W, mu, Xv, p0v)
        ref, tol = orc.gemv(W.w_hat, xm), orc.tolerance(W.w_hat, xm)
        y = Y.cpu().numpy().astype(np.float64)
        assert np.isfinite(y).all() and (np.abs(y - ref) <= tol).all()
        single = _run(W, mu, Xd, p0d, M)
        assert torch.equal(single, Y)


def test_prefill_grouped_rejects_bad_groups():
    W = H.pack_sq(H.random_sq_codes(450, 256, 512))
    M = 64
    _, Xd = _bf16(inputs.gen_activation(451, M, 512, n_outliers=8))
    Y = torch.zeros((M, 256), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.rwkvq_prefill_workspace_bytes(W.desc, M, False), dtype=torch.uint8, device="cuda")
    e = dict(desc=W.desc, W=W.dev, X=Xd, Y=Y, workspace=ws)
    with pytest.raises(B.RwkvqError):
        B.rwkvq_gemm_prefill_grouped([e, dict(e)], M)                 # shared output and workspace
    with pytest.raises(B.RwkvqError):
        B.rwkvq_gemm_prefill_grouped([dict(e, workspace=ws[:1024])], M)      # workspace too small
    with pytest.raises(B.RwkvqError):
        B.rwkvq_gemm_prefill_grouped([e] * 17, M)
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 0
