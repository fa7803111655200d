"""GPU parity of the decode path against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _dequant(P, dtype=torch.float32):
    shape = (P.ic,) if P.oc == 1 else (P.oc, P.ic)
    out = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
    B.rwkvq_dequant(P.desc, P.dev, out)
    torch.cuda.synchronize()
    return out


def _check_decode_exact(P):
    got = _dequant(P).double().cpu().numpy()
    assert np.array_equal(got, P.w_hat.reshape(got.shape)), "decoded weights are not bit-exact"
    got16 = _dequant(P, torch.bfloat16).float().cpu().numpy()
    assert np.array_equal(got16, orc.bf16_rne(P.w_hat.reshape(got16.shape)))


def _check_gemv(W, mu, x16, xp16, y_dtype=torch.float32):
    y = H.run_gemv(W, mu, x16, xp16, y_dtype)
    ref, tol = H.reference(W, mu, x16, xp16)
    err = np.abs(y - ref)
    if y_dtype == torch.float16:
        tol = tol + np.abs(ref) * 2.0 ** -10
    ratio = float((err / np.maximum(tol, 1e-300)).max())
    assert np.isfinite(y).all() and (err <= tol).all(), f"max err/tol = {ratio}"
    return ratio


@pytest.fixture(scope="module")
def config1():
    """Single 512x512 N(0, 0.02) matrix, seed 0, quantized twice by the oracle: 3-bit g128 SQ and
    2-D VQ with a 64-entry codebook per 256x256 tile (k-means++, 10 Lloyd iterations); a 512-long
    mu vector VQ-coded the same way; batch-1 fp16 N(0,1) activations."""
    w = inputs.gen_weight(0, 512, 512, "gauss")
    q, s, z = orc.sq_encode(w)
    cbs, idx = orc.vq_encode(w, entries=64, tile=256, iters=10, seed=0)
    mu = inputs.gen_mu(1, 512)
    mcb, mix = orc.mu_encode(mu, entries=64, iters=10, seed=0)
    x, xp = inputs.gen_activation_pair(2, 1, 512, n_outliers=0)
    return dict(sq=H.pack_sq(dict(q=q, scale=s, zero=z)), vq=H.pack_vq(dict(q=idx, codebook=cbs), 6),
                mu=H.pack_mu(dict(q=mix, codebook=mcb)), x=x.astype(np.float16), xp=xp.astype(np.float16), w=w)


def test_config1_decode_bit_exact(config1):
    _check_decode_exact(config1["sq"])
    _check_decode_exact(config1["vq"])
    _check_decode_exact(config1["mu"])
    # the quantizers did their job: reconstruction error is small relative to the weights
    w = config1["w"].astype(np.float64)
    for k in ("sq", "vq"):
        rel = np.linalg.norm(config1[k].w_hat - w) / np.linalg.norm(w)
        assert rel < 0.3


def test_config1_gemv_with_fused_token_shift(config1):
    for k in ("sq", "vq"):
        _check_gemv(config1[k], config1["mu"], config1["x"], config1["xp"])
        _check_gemv(config1[k], None, config1["x"], None)


def test_one_hot_probes_read_back_decoded_columns(config1):
    # x = e_j through the product returns column j of the decoded matrix
    for k in ("sq", "vq"):
        W = config1[k]
        cols = [0, 1, 2, 3, 127, 128, 255, 256, 300, 511]
        x = np.zeros((len(cols), 512), np.float16)
        for b, c in enumerate(cols):
            x[b, c] = 1.0
        y = H.run_gemv(W, None, x, None)
        ref = W.w_hat[:, cols].T
        assert np.abs(y - ref).max() <= 2e-3 * np.sqrt((W.w_hat ** 2).sum(axis=1)).max()
        if k == "vq":
            assert np.array_equal(y, ref)        # table lookup times 1.0 is exact


@pytest.mark.parametrize("oc,ic", [(16, 128), (48, 384), (128, 256), (2048, 2048), (1024, 7168), (7168, 2048)])
@pytest.mark.parametrize("Bn", [1, 3, 8, 9, 16])
def test_sq_shapes_and_batches(oc, ic, Bn):
    W = H.pack_sq(H.random_sq_codes(oc * 7 + ic, oc, ic))
    if Bn == 1:
        _check_decode_exact(W)
    x, xp = inputs.gen_activation_pair(Bn + ic, Bn, ic, n_outliers=8)
    mu = H.pack_mu(H.random_mu_codes(ic, ic)) if Bn in (1, 8, 16) else None
    _check_gemv(W, mu, x.astype(np.float16), xp.astype(np.float16))


@pytest.mark.parametrize("bits", [6, 8])
@pytest.mark.parametrize("oc,ic", [(256, 256), (512, 768), (2048, 2048), (1024, 7168)])
@pytest.mark.parametrize("Bn", [1, 5, 8, 16])
def test_vq_shapes_and_batches(bits, oc, ic, Bn):
    W = H.pack_vq(H.random_vq_codes(oc * 3 + ic + bits, oc, ic, bits), bits)
    if Bn == 1:
        _check_decode_exact(W)
    x, xp = inputs.gen_activation_pair(Bn + ic, Bn, ic, n_outliers=8)
    mu = H.pack_mu(H.random_mu_codes(ic + 1, ic, bits), bits) if Bn in (1, 16) else None
    _check_gemv(W, mu, x.astype(np.float16), xp.astype(np.float16))


def test_fp16_output_and_zero_input():
    W = H.pack_sq(H.random_sq_codes(77, 256, 512))
    x, xp = inputs.gen_activation_pair(5, 4, 512)
    _check_gemv(W, None, x.astype(np.float16), None, torch.float16)
    y = H.run_gemv(W, None, np.zeros((2, 512), np.float16), None)
    assert np.array_equal(y, np.zeros((2, 256)))


def test_constant_codebook_gives_constant_matrix_product():
    # every codebook entry equal -> decoded matrix is constant -> y = c_even*sum(x_even) + c_odd*sum(x_odd)
    codes = H.random_vq_codes(3, 256, 512, 6)
    codes["codebook"][...] = np.array([0.5, -0.25], np.float16)
    W = H.pack_vq(codes, 6)
    x = np.arange(512, dtype=np.float64).reshape(1, 512) % 7 - 3
    y = H.run_gemv(W, None, x.astype(np.float16), None)
    expect = 0.5 * x[0, 0::2].sum() - 0.25 * x[0, 1::2].sum()
    assert np.array_equal(y, np.full((1, 256), expect))


def test_mu_special_values_select_x_or_xprev():
    W = H.pack_sq(H.random_sq_codes(8, 128, 256))
    x, xp = inputs.gen_activation_pair(9, 2, 256)
    x16, xp16 = x.astype(np.float16), xp.astype(np.float16)
    for val, src in ((0.0, x16), (1.0, xp16)):
        mc = H.random_mu_codes(1, 256)
        mc["codebook"][...] = np.float16(val)
        y_mix = H.run_gemv(W, H.pack_mu(mc), x16, xp16)
        y_plain = H.run_gemv(W, None, src, None)
        assert np.array_equal(y_mix, y_plain)


def test_argument_errors_are_reported_before_launch():
    W = H.pack_sq(H.random_sq_codes(8, 128, 256))
    x = torch.zeros((1, 256), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 128), dtype=torch.float32, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemv(W.desc, W.dev, None, None, x, None, 17, y, ws)
    assert e.value.status == 1
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemv(W.desc, W.dev[8:], None, None, x, None, 1, y, ws)
    assert e.value.status == 3
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemv(W.desc, W.dev, None, None, x, None, 1, y, ws[:16])
    assert e.value.status == 5
    mu = H.pack_mu(H.random_mu_codes(1, 512))
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemv(W.desc, W.dev, mu.desc, mu.dev, x, x, 1, y, ws)
    assert e.value.status == 2
    assert B.rwkvq_device_status() == 0


def _extreme_sq_codes(seed, oc, ic):
    """Valid logical SQ codes whose scales cover the whole fp16 range (subnormals, the smallest
    subnormal 2^-24, scales of 2^15 and above) and whose zero points include non-integers: Eq. 2's
    decode s * (q - z) is defined for all of them (two fp32 operations, no FMA contraction)."""
    rng = np.random.default_rng(seed)
    codes = H.random_sq_codes(seed, oc, ic)
    s = codes["scale"].astype(np.float64)
    pick = [2.0 ** -24, 3 * 2.0 ** -24, 2.0 ** -15, 6.0e-5, 2.0 ** 15, 40000.0, 65504.0, 1.0, 0.013]
    s[:] = rng.choice(pick, size=s.shape)
    codes["scale"] = s.astype(np.float16)
    z = codes["zero"].astype(np.float64)
    frac = rng.random(z.shape) < 0.3
    z[frac] = rng.choice([0.5, 2.25, 3.125, 6.75, 0.0009765625], size=int(frac.sum()))
    codes["zero"] = z.astype(np.float16)
    return codes


@pytest.mark.parametrize("oc,ic,Bn", [(64, 512, 1), (256, 1024, 8), (128, 2048, 16)])
def test_sq_extreme_scales_and_fractional_zero_points(oc, ic, Bn):
    W = H.pack_sq(_extreme_sq_codes(oc + ic + Bn, oc, ic))
    s = W.codes["scale"].astype(np.float64)
    assert (s < 6.2e-5).any() and (s >= 2.0 ** 15).any()               # subnormal and very large scales are present
    assert (W.codes["zero"].astype(np.float64) % 1 != 0).any()          # and zero points that are no integers
    _check_decode_exact(W)
    # Scales this far apart make rows that differ by ten orders of magnitude: activations with a
    # few large channels exercise the fp32 accumulation of the per-group terms.
    x, xp = inputs.gen_activation_pair(Bn + ic, Bn, ic, n_outliers=8)
    mu = H.pack_mu(H.random_mu_codes(ic, ic)) if Bn != 8 else None
    _check_gemv(W, mu, x.astype(np.float16), xp.astype(np.float16))
