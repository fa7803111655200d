"""Device quantizers (rwkvq_quantize_dev, rwkvq_calib_representative) against the oracle.

SQ (Section 3.2 Eq. 2): codes, scales and zero points bit-exact, image payload identical to the host
packer's.  VQ (Eq. 3) and the weighted k-means of Section 4.2: codebook values have several correct
answers, so what is unique is compared exactly (the assignment given the codebook, zero error on few
distinct vectors) and the rest through the loss the method minimises, next to the oracle's own run.
"""
import numpy as np
import pytest
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B

pytestmark = pytest.mark.gpu


def quantize_dev(w16, method, bits, elem_weight=None, seed=0, iters=10):
    oc, ic = (1, w16.shape[0]) if w16.ndim == 1 else w16.shape
    d0 = B.rwkvq_desc_for(oc, ic, method, bits)
    wd = torch.from_numpy(np.ascontiguousarray(w16)).cuda()
    img = torch.full((int(d0.image_bytes),), 0xAB, dtype=torch.uint8, device="cuda")
    ws = torch.empty(B.rwkvq_quantize_workspace_bytes(), dtype=torch.uint8, device="cuda")
    ew = None if elem_weight is None else torch.from_numpy(np.ascontiguousarray(elem_weight, dtype=np.float32)).cuda()
    d = B.rwkvq_quantize_dev(wd, oc, ic, method, bits, img, ws, elem_weight=ew, kmeans_iters=iters, seed=seed)
    torch.cuda.synchronize()
    assert d.image_bytes == d0.image_bytes
    return d, img


def sq_cases():
    rng = np.random.default_rng(42)
    out = {}
    out["gauss_512"] = (rng.standard_normal((512, 512)) * 0.02).astype(np.float16)
    out["ragged_272x384"] = (rng.standard_normal((272, 384)) * 0.02).astype(np.float16)
    out["student_1024x768"] = (rng.standard_t(3, (1024, 768)) * 0.01).astype(np.float16)
    w = (rng.standard_normal((256, 1024)) * 0.02).astype(np.float16)
    w[0, :128] = 0.0                       # constant groups: zero, positive, negative
    w[1, :128] = 0.375
    w[2, 128:256] = -0.0625
    w[3, :128] = np.float16(6e-8)          # subnormal constant
    w[4, :128] = np.where(np.arange(128) % 2 == 0, np.float16(6e-8), np.float16(1.2e-7))   # scale underflows to 0
    w[5, :128] = (100.0 + rng.uniform(0, 0.5, 128)).astype(np.float16)                      # far from zero: z saturates
    w[6, :128] = (np.arange(128) % 15) * 0.5                                                # s = 1: quotients on ties
    w[7, :128] = -((np.arange(128) % 15) * 0.5)
    w[8, :128] = (np.arange(128) % 8).astype(np.float16) * np.float16(0.1)                  # ramp: q = t
    w[9, :128] = rng.choice([-60000.0, 60000.0, 1e-4], 128)                                # full fp16 range
    w[10, 896:1024] = rng.uniform(-1, 1, 128) * 2.0 ** -14                                  # around the subnormal boundary
    out["special_256x1024"] = w
    return out


@pytest.mark.parametrize("name", list(sq_cases().keys()))
def test_sq_device_quantizer_is_bit_exact(name):
    w16 = sq_cases()[name]
    oc, ic = w16.shape
    d, img = quantize_dev(w16, B.RWKVQ_SQ, 3)
    host = img.cpu().numpy()
    d2, codes = B.rwkvq_image_unpack(host)
    q, s, z = orc.sq_encode(w16)
    assert (d2.oc, d2.ic, d2.method, d2.bits) == (oc, ic, B.RWKVQ_SQ, 3)
    assert np.array_equal(np.asarray(codes["q"]).reshape(oc, ic), q)
    assert np.array_equal(np.asarray(codes["scale"]).view(np.uint16).reshape(s.shape), s.view(np.uint16))
    # zero points are compared as numbers: a group whose minimum is 0 gets z = -0.0 from the oracle's
    # round(-min / s) and +0.0 from a clamp written with max(); both denote the same zero point
    assert np.array_equal(np.asarray(codes["zero"]).reshape(z.shape).astype(np.float64), z.astype(np.float64))
    # the whole payload (padding included) equals the host packer's
    ref = B.rwkvq_pack(w16, oc, ic, B.RWKVQ_SQ, 3).image()
    assert np.array_equal(host[256:], ref[256:])      # (both write +0.0 for such a zero point)


def test_sq_device_image_feeds_the_products():
    rng = np.random.default_rng(3)
    w16 = (rng.standard_normal((512, 768)) * 0.02).astype(np.float16)
    d, img = quantize_dev(w16, B.RWKVQ_SQ, 3)
    q, s, z = orc.sq_encode(w16)
    w_hat = orc.sq_decode(q, s, z)
    out = torch.empty((512, 768), dtype=torch.float32, device="cuda")
    B.rwkvq_dequant(d, img, out)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), w_hat.astype(np.float32).astype(np.float64))
    x = rng.standard_normal((3, 768)).astype(np.float16)
    y = torch.empty((3, 512), dtype=torch.float32, device="cuda")
    ws = torch.zeros(max(256, B.rwkvq_gemv_workspace_bytes(d, 3)), dtype=torch.uint8, device="cuda")
    B.rwkvq_gemv(d, img, None, None, torch.from_numpy(x).cuda(), None, 3, y, ws)
    torch.cuda.synchronize()
    ref = orc.gemv(w_hat, x.astype(np.float64))
    tol = orc.tolerance(w_hat, x.astype(np.float64))
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref) <= tol)


def test_sq_device_image_of_special_groups_feeds_the_products():
    # the matrix of degenerate groups (constants, +-0, the full fp16 range, subnormals): its device
    # image must decode to the oracle's values bit for bit and multiply within the tolerance
    w16 = sq_cases()["special_256x1024"]
    oc, ic = w16.shape
    d, img = quantize_dev(w16, B.RWKVQ_SQ, 3)
    q, s, z = orc.sq_encode(w16)
    w_hat = orc.sq_decode(q, s, z)
    out = torch.empty((oc, ic), dtype=torch.float32, device="cuda")
    B.rwkvq_dequant(d, img, out)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), w_hat)
    rng = np.random.default_rng(12)
    for Bn in (1, 5):
        x = rng.standard_normal((Bn, ic)).astype(np.float16)
        y = torch.empty((Bn, oc), dtype=torch.float32, device="cuda")
        ws = torch.zeros(max(256, B.rwkvq_gemv_workspace_bytes(d, Bn)), dtype=torch.uint8, device="cuda")
        B.rwkvq_gemv(d, img, None, None, torch.from_numpy(x).cuda(), None, Bn, y, ws)
        torch.cuda.synchronize()
        ref = orc.gemv(w_hat, x.astype(np.float64))
        tol = orc.tolerance(w_hat, x.astype(np.float64))
        got = y.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all() and np.all(np.abs(got - ref) <= tol)


def tile_vectors(w16, tr, tc):
    return w16[tr * 256:(tr + 1) * 256, tc * 256:(tc + 1) * 256].astype(np.float64).reshape(-1, 2)


@pytest.mark.parametrize("bits,oc,ic", [(6, 512, 768), (8, 256, 512)])
def test_vq_device_quantizer_valid_and_as_good_as_the_oracle(bits, oc, ic):
    rng = np.random.default_rng(10 + bits)
    E = 1 << bits
    w16 = (rng.standard_t(3, (oc, ic)) * 0.01).astype(np.float16)
    d, img = quantize_dev(w16, B.RWKVQ_VQ, bits, seed=5)
    _, img_again = quantize_dev(w16, B.RWKVQ_VQ, bits, seed=5)
    assert torch.equal(img, img_again), "the device quantizer is not reproducible"
    _, codes = B.rwkvq_image_unpack(img.cpu().numpy())
    cbs = np.asarray(codes["codebook"]).reshape(oc // 256, ic // 256, E, 2)
    idx = np.asarray(codes["q"]).reshape(oc, ic // 2)
    assert np.isfinite(cbs.astype(np.float64)).all()
    cb_o, idx_o = orc.vq_encode(w16, entries=E, seed=5)
    mse_dev = mse_orc = 0.0
    for tr in range(oc // 256):
        for tc in range(ic // 256):
            v = tile_vectors(w16, tr, tc)
            c = cbs[tr, tc].astype(np.float64)
            ix = idx[tr * 256:(tr + 1) * 256, tc * 128:(tc + 1) * 128].reshape(-1)
            # unique given the codebook: nearest centre, lowest index on ties (Eq. 3)
            assert np.array_equal(ix, orc._nearest(v, c))
            mse_dev += float(((v - c[ix]) ** 2).sum())
            co = cb_o[tr, tc].astype(np.float64)
            io = idx_o[tr * 256:(tr + 1) * 256, tc * 128:(tc + 1) * 128].reshape(-1)
            mse_orc += float(((v - co[io]) ** 2).sum())
    assert mse_dev <= 1.10 * mse_orc, (mse_dev, mse_orc)
    # the image is what the products read
    out = torch.empty((oc, ic), dtype=torch.float32, device="cuda")
    B.rwkvq_dequant(d, img, out)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), orc.vq_decode(cbs, idx))


def test_vq_device_lloyd_iterations_lower_the_loss():
    rng = np.random.default_rng(2)
    w16 = (rng.standard_normal((256, 256)) * 0.02).astype(np.float16)
    v = tile_vectors(w16, 0, 0)
    losses = []
    for iters in (0, 1, 3, 10):
        _, img = quantize_dev(w16, B.RWKVQ_VQ, 6, seed=9, iters=iters)
        _, codes = B.rwkvq_image_unpack(img.cpu().numpy())
        c = np.asarray(codes["codebook"]).reshape(64, 2).astype(np.float64)
        losses.append(float(((v - c[np.asarray(codes["q"]).reshape(-1)]) ** 2).sum()))
    assert losses[1] < losses[0] and losses[2] < losses[1] and losses[3] < losses[2]


@pytest.mark.parametrize("bits", [6, 8])
def test_vq_device_zero_error_on_few_distinct_vectors(bits):
    rng = np.random.default_rng(1)
    E = 1 << bits
    protos = (rng.standard_normal((E - 3, 2)) * 0.05).astype(np.float16)
    pick = rng.integers(0, len(protos), (256, 128))
    w16 = protos[pick].reshape(256, 256)
    _, img = quantize_dev(w16, B.RWKVQ_VQ, bits, seed=1)
    _, codes = B.rwkvq_image_unpack(img.cpu().numpy())
    w_hat = orc.vq_decode(np.asarray(codes["codebook"]).reshape(1, 1, E, 2), np.asarray(codes["q"]).reshape(256, 128))
    assert np.array_equal(w_hat, w16.astype(np.float64))
    const = np.full((256, 512), np.float16(-0.3125))
    _, img = quantize_dev(const, B.RWKVQ_VQ, bits)
    _, codes = B.rwkvq_image_unpack(img.cpu().numpy())
    w_hat = orc.vq_decode(np.asarray(codes["codebook"]).reshape(1, 2, E, 2), np.asarray(codes["q"]).reshape(256, 256))
    assert np.array_equal(w_hat, const.astype(np.float64))


def calib_samples(S, n, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((S, n)) * (1.0 + 4.0 * (rng.random(n) < 0.05))[None, :] + rng.standard_normal(n)[None, :] * 0.5
    hot = rng.random((S, n)) < 0.01
    x[hot] *= 20.0
    return x.astype(np.float32)


@pytest.mark.parametrize("S,n,pct", [(128, 2048, 1.0), (128, 1000, 5.0), (101, 70, 10.0), (16, 33, 0.0), (7, 5, 25.0)])
def test_representative_activation_matches_oracle(S, n, pct):
    x = calib_samples(S, n, S + n)
    xd = torch.from_numpy(x).cuda()
    rep = torch.empty(n, dtype=torch.float32, device="cuda")
    rsq = torch.empty(n, dtype=torch.float32, device="cuda")
    B.rwkvq_calib_representative(xd, pct, rep, rsq)
    torch.cuda.synchronize()
    ref = orc.representative_activation(x.astype(np.float64), pct)
    got = rep.cpu().numpy().astype(np.float64)
    # fp64 mean in another summation order, then one rounding to fp32
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -23 + 1e-12)
    assert np.all(np.abs(rsq.cpu().numpy().astype(np.float64) - ref * ref) <= ref * ref * 2.0 ** -22 + 1e-12)


@pytest.mark.parametrize("ic,bits", [(2048, 6), (4096, 6), (5120, 8)])
def test_weighted_mu_quantizer(ic, bits):
    rng = np.random.default_rng(ic)
    E = 1 << bits
    mu16 = rng.uniform(0.0, 1.0, ic).astype(np.float16)
    x = calib_samples(128, ic, 7)
    rep = orc.representative_activation(x.astype(np.float64), 1.0)
    xd = torch.from_numpy(x).cuda()
    rsq = torch.empty(ic, dtype=torch.float32, device="cuda")
    B.rwkvq_calib_representative(xd, 1.0, None, rsq)
    torch.cuda.synchronize()
    wts = rsq.cpu().numpy()
    assert np.all(np.abs(wts.astype(np.float64) - rep * rep) <= rep * rep * 2.0 ** -22 + 1e-12)
    v = mu16.astype(np.float64).reshape(-1, 2)
    w2 = wts.astype(np.float64).reshape(-1, 2)

    def loss_of(img):
        _, codes = B.rwkvq_image_unpack(img.cpu().numpy())
        c = np.asarray(codes["codebook"]).reshape(E, 2).astype(np.float64)
        ix = np.asarray(codes["q"]).reshape(-1)
        return c, ix, float((w2 * (v - c[ix]) ** 2).sum())

    d, img = quantize_dev(mu16, B.RWKVQ_VQ, bits, elem_weight=wts, seed=3)
    c, ix, loss_w = loss_of(img)
    assert np.array_equal(ix, orc._nearest(v, c, w2))          # unique given the codebook (Eq. 19)
    loss_o = 0.0
    for sd in (3, 4, 5):      # the oracle's own spread over seeds is of the order of ten per cent
        cb_o, ix_o = orc.mu_encode(mu16, entries=E, seed=sd, act_sq=wts.astype(np.float64))
        loss_o += float((w2 * (v - cb_o.astype(np.float64)[ix_o]) ** 2).sum()) / 3.0
    assert loss_w <= 1.35 * loss_o, (loss_w, loss_o)
    # the plain codebook of the same vector is worse under Eq. 19
    _, img_plain = quantize_dev(mu16, B.RWKVQ_VQ, bits, seed=3)
    c_p, ix_p, loss_p = loss_of(img_plain)
    assert np.array_equal(ix_p, orc._nearest(v, c_p))
    assert loss_w < loss_p
    # the image decodes to the codebook entries
    out = torch.empty(ic, dtype=torch.float32, device="cuda")
    B.rwkvq_dequant(d, img, out)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), orc.mu_decode(c.astype(np.float16), ix))


def test_quantize_dev_error_paths():
    w = torch.zeros((256, 256), dtype=torch.float16, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    d0 = B.rwkvq_desc_for(256, 256, B.RWKVQ_SQ, 3)
    img = torch.empty(int(d0.image_bytes) + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_quantize_dev(w, 256, 256, B.RWKVQ_SQ, 3, img[:1024], ws)
    assert e.value.status == 5
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_quantize_dev(w, 256, 256, B.RWKVQ_SQ, 3, img[16:], ws)
    assert e.value.status == 3
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_quantize_dev(w, 250, 256, B.RWKVQ_SQ, 3, img, ws)
    assert e.value.status == 2
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_quantize_dev(w, 256, 256, B.RWKVQ_VQ, 6, img, ws, elem_weight=torch.ones(256, device="cuda"))
    assert e.value.status == 1
    for method, bits in ((B.RWKVQ_SQ, 3), (B.RWKVQ_VQ, 6)):
        bad = torch.zeros((256, 256), dtype=torch.float16, device="cuda")
        bad[200, 131] = float("nan")
        with pytest.raises(B.RwkvqError) as e:
            B.rwkvq_quantize_dev(bad, 256, 256, method, bits, img, ws)
        assert e.value.status == 4
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_calib_representative(torch.zeros((1, 8), device="cuda"), 1.0, torch.zeros(8, device="cuda"))
    assert e.value.status == 1


@pytest.mark.parametrize("method,bits,oc,ic", [(B.RWKVQ_SQ, 3, 272, 384), (B.RWKVQ_SQ, 3, 512, 512), (B.RWKVQ_VQ, 6, 256, 512),
                                               (B.RWKVQ_VQ, 8, 256, 256)])
def test_quant_error_matches_oracle(method, bits, oc, ic):
    rng = np.random.default_rng(oc + ic + bits)
    w16 = (rng.standard_t(3, (oc, ic)) * 0.01).astype(np.float16)
    d, img = quantize_dev(w16, method, bits, seed=2, iters=3)
    _, codes = B.rwkvq_image_unpack(img.cpu().numpy())
    if method == B.RWKVQ_SQ:
        w_hat = orc.sq_decode(np.asarray(codes["q"]).reshape(oc, ic), np.asarray(codes["scale"]), np.asarray(codes["zero"]))
    else:
        w_hat = orc.vq_decode(np.asarray(codes["codebook"]).reshape(oc // 256, ic // 256, 1 << bits, 2),
                              np.asarray(codes["q"]).reshape(oc, ic // 2))
    wd = torch.from_numpy(w16).cuda()
    sse = B.rwkvq_quant_error(wd, d, img)
    ref = orc.quant_sse(w16, w_hat)
    assert abs(sse - ref) <= 1e-12 * ref
    assert sse == B.rwkvq_quant_error(wd, d, img)          # reproducible


def test_mse_selector_picks_the_smaller_error():
    # Section 5.3's "MSE" selector: code the matrix both ways, keep the coding with the smaller error
    rng = np.random.default_rng(77)
    for kind in ("gauss", "student"):
        w16 = ((rng.standard_normal((256, 512)) * 0.02) if kind == "gauss" else rng.standard_t(3, (256, 512)) * 0.01).astype(np.float16)
        wd = torch.from_numpy(w16).cuda()
        dq, iq = quantize_dev(w16, B.RWKVQ_SQ, 3)
        dv, iv = quantize_dev(w16, B.RWKVQ_VQ, 6, seed=1)
        e_sq, e_vq = B.rwkvq_quant_error(wd, dq, iq), B.rwkvq_quant_error(wd, dv, iv)
        q, s, z = orc.sq_encode(w16)
        assert abs(e_sq - orc.quant_sse(w16, orc.sq_decode(q, s, z))) <= 1e-12 * e_sq
        assert e_sq > 0.0 and e_vq > 0.0 and (e_sq < e_vq) == (orc.quant_sse(w16, orc.sq_decode(q, s, z)) < e_vq)


def test_async_quantizer_and_check():
    rng = np.random.default_rng(9)
    ws = torch.zeros(B.rwkvq_quantize_workspace_bytes(), dtype=torch.uint8, device="cuda")
    mats = [(rng.standard_normal((256, 384)) * 0.02).astype(np.float16) for _ in range(3)]
    imgs = []
    for w16 in mats:
        d0 = B.rwkvq_desc_for(256, 384, B.RWKVQ_SQ, 3)
        img = torch.empty(int(d0.image_bytes), dtype=torch.uint8, device="cuda")
        B.rwkvq_quantize_dev_async(torch.from_numpy(w16).cuda(), 256, 384, B.RWKVQ_SQ, 3, img, ws)
        imgs.append(img)
    assert B.rwkvq_quantize_check(ws) == 0
    for w16, img in zip(mats, imgs):
        ref = B.rwkvq_pack(w16, 256, 384, B.RWKVQ_SQ, 3).image()
        assert np.array_equal(img.cpu().numpy()[256:], ref[256:])
    bad = mats[1].copy()
    bad[7, 300] = np.float16(np.inf)
    for w16 in (mats[0], bad, mats[2]):           # the flag of the middle call survives the later one
        B.rwkvq_quantize_dev_async(torch.from_numpy(w16).cuda(), 256, 384, B.RWKVQ_SQ, 3, imgs[0], ws)
    assert B.rwkvq_quantize_check(ws) == 4
    assert B.rwkvq_quantize_check(ws) == 0        # cleared by the check
