"""Host-side tests of the C-ABI library: symbols, quantizers, bit packing, error paths.
No compute call touches a GPU here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import build as build_mod
from paper_2505_03803_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "rwkvq.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(rwkvq_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations parsed"
    lib = C.CDLL(B.LIB_PATH)
    missing = [n for n in sorted(declared) if not hasattr(lib, n)]
    assert not missing, f"declared but not exported: {missing}"
    assert set(B.EXPORTS) == declared


def test_sq_encoder_matches_oracle_codes_exactly():
    for seed, kind in ((0, "gauss"), (1, "student"), (2, "uniform")):
        w = inputs.gen_weight(seed, 64, 512, kind)
        w[3, 128:256] = np.float16(0.0)         # degenerate groups
        w[5, 0:128] = np.float16(-0.375)
        w[7, 256:384] = np.float16(0.011)
        blob = B.rwkvq_pack(w, 64, 512, B.RWKVQ_SQ, 3)
        got = blob.export_codes()
        q, s, z = orc.sq_encode(w)
        assert np.array_equal(got["q"], q)
        assert np.array_equal(got["scale"].view(np.uint16), s.view(np.uint16))
        assert np.array_equal(got["zero"].view(np.uint16), z.view(np.uint16))


def _spec_sq_image_payload(q, s, z, oc, ic):
    """Bit layout of the SQ payload written from the format description, independent of the C++ packer."""
    oc_pad, ic_pad = -(-oc // 128) * 128, -(-ic // 256) * 256
    MB, KT, ng = oc_pad // 128, ic_pad // 256, ic // 128
    out = np.zeros(MB * KT * 8 * 1664, np.uint8)
    words = out.view(np.uint32)
    su, zu = s.view(np.uint16), z.view(np.uint16)
    for mb in range(MB):
        for kt in range(KT):
            for rt in range(8):
                base = ((mb * KT + kt) * 8 + rt) * 1664
                for L in range(32):
                    g, t = L >> 2, L & 3
                    for i in range(4):
                        for e in range(16):
                            m, R = e >> 2, e & 3
                            row = mb * 128 + rt * 16 + g + 8 * (R & 1)
                            col = kt * 256 + 64 * i + 16 * m + 4 * t + 2 * (R >> 1)
                            for hf in range(2):
                                code = int(q[row, col + hf]) if (row < oc and col + hf < ic) else 0
                                if e < 15:
                                    widx = 3 * i + e // 5
                                    wpos = (base + (widx >> 2) * 512 + L * 16 + (widx & 3) * 4) // 4
                                    words[wpos] |= np.uint32(code << (16 * hf + 3 * (e % 5)))
                                else:
                                    for b in range(3):
                                        widx = 3 * i + b
                                        wpos = (base + (widx >> 2) * 512 + L * 16 + (widx & 3) * 4) // 4
                                        words[wpos] |= np.uint32(((code >> b) & 1) << (16 * hf + 15))
                sz = out[base + 1536: base + 1664].view(np.uint16)
                for g in range(8):
                    for k in range(4):
                        row, grp = mb * 128 + rt * 16 + g + 8 * (k >> 1), kt * 2 + (k & 1)
                        if row < oc and grp < ng:
                            sz[g * 8 + 2 * k] = su[row, grp]
                            sz[g * 8 + 2 * k + 1] = zu[row, grp]
    return out


def test_sq_image_matches_layout_spec_and_roundtrips():
    rng = np.random.default_rng(3)
    oc, ic = 48, 384          # exercises row padding to 128 and column padding to 256
    q = rng.integers(0, 8, size=(oc, ic), dtype=np.uint8)
    s = rng.random((oc, ic // 128)).astype(np.float16)
    z = rng.integers(0, 8, size=(oc, ic // 128)).astype(np.float16)
    blob = B.rwkvq_pack(None, oc, ic, B.RWKVQ_SQ, 3, codes=dict(q=q, scale=s, zero=z))
    img = blob.image()
    d = blob.desc
    assert (d.oc_pad, d.ic_pad) == (128, 512)
    assert d.image_bytes == 256 + 1 * 2 * 8 * 1664 == img.nbytes
    assert np.array_equal(img[256:], _spec_sq_image_payload(q, s, z, oc, ic))
    d2, codes = B.rwkvq_image_unpack(img)
    assert (d2.oc, d2.ic, d2.method, d2.bits) == (oc, ic, B.RWKVQ_SQ, 3)
    assert np.array_equal(codes["q"], q)
    assert np.array_equal(codes["scale"].view(np.uint16), s.view(np.uint16))
    assert np.array_equal(codes["zero"].view(np.uint16), z.view(np.uint16))


def _spec_vq_payload(idx, oc, ic, bits):
    MB, KT = oc // 128, ic // 256
    rb = 64 * 32 * bits // 8
    out = np.zeros(MB * KT * 8 * rb, np.uint8)
    for mb in range(MB):
        for kt in range(KT):
            for rt in range(8):
                base = ((mb * KT + kt) * 8 + rt) * rb
                for L in range(32):
                    g, t = L >> 2, L & 3
                    stream = 0
                    for n in range(64):
                        j, R = n >> 2, n & 3
                        row = mb * 128 + rt * 16 + g + 8 * (R & 1)
                        pair = kt * 128 + 8 * j + 2 * t + (R >> 1)
                        stream |= int(idx[row, pair]) << (bits * n)
                    for widx in range(2 * bits):
                        word = (stream >> (32 * widx)) & 0xFFFFFFFF
                        off = base + (widx >> 2) * 512 + L * 16 + (widx & 3) * 4
                        out[off:off + 4] = np.frombuffer(np.uint32(word).tobytes(), np.uint8)
    return out


@pytest.mark.parametrize("bits", [6, 8])
def test_vq_image_matches_layout_spec_and_roundtrips(bits):
    rng = np.random.default_rng(4 + bits)
    oc, ic, E = 256, 512, 1 << bits
    idx = rng.integers(0, E, size=(oc, ic // 2), dtype=np.uint8)
    cb = rng.standard_normal((1, 2, E, 2)).astype(np.float16)
    blob = B.rwkvq_pack(None, oc, ic, B.RWKVQ_VQ, bits, codes=dict(q=idx, codebook=cb))
    img = blob.image()
    d = blob.desc
    rb = 64 * 32 * bits // 8
    npay = 2 * 2 * 8 * rb
    assert d.stream_bytes == npay + 2 * E * 4
    assert np.array_equal(img[256:256 + npay], _spec_vq_payload(idx, oc, ic, bits))
    assert np.array_equal(img[256 + npay:256 + npay + 2 * E * 4].view(np.uint16), cb.view(np.uint16).reshape(-1))
    _, codes = B.rwkvq_image_unpack(img)
    assert np.array_equal(codes["q"], idx)
    assert np.array_equal(codes["codebook"].view(np.uint16), cb.view(np.uint16))


@pytest.mark.parametrize("bits", [6, 8])
def test_vector_image_roundtrip(bits):
    rng = np.random.default_rng(9)
    ic, E = 514, 1 << bits
    idx = rng.integers(0, E, size=(ic // 2,), dtype=np.uint8)
    cb = rng.random((E, 2)).astype(np.float16)
    blob = B.rwkvq_pack(None, 1, ic, B.RWKVQ_VQ, bits, codes=dict(q=idx, codebook=cb))
    img = blob.image()
    # natural-order little-endian bit stream
    stream = 0
    for p in range(ic // 2):
        stream |= int(idx[p]) << (bits * p)
    nbytes = (ic // 2 * bits + 7) // 8
    assert bytes(img[256:256 + nbytes]) == stream.to_bytes(nbytes, "little")
    _, codes = B.rwkvq_image_unpack(img)
    assert np.array_equal(codes["q"], idx) and np.array_equal(codes["codebook"].view(np.uint16), cb.view(np.uint16))


def test_bytes_per_weight():
    w = inputs.gen_weight(0, 256, 512)
    sq = B.rwkvq_pack(w, 256, 512, B.RWKVQ_SQ, 3).desc
    assert sq.stream_bytes / (256 * 512) == 0.40625            # 3.25 bits per weight
    q = np.zeros((256, 256), np.uint8)
    v6 = B.rwkvq_pack(None, 256, 512, B.RWKVQ_VQ, 6, codes=dict(q=q, codebook=np.zeros((1, 2, 64, 2), np.float16))).desc
    v8 = B.rwkvq_pack(None, 256, 512, B.RWKVQ_VQ, 8, codes=dict(q=q, codebook=np.zeros((1, 2, 256, 2), np.float16))).desc
    assert v6.stream_bytes / (256 * 512) == 0.37890625
    assert v8.stream_bytes / (256 * 512) == 0.515625


@pytest.mark.parametrize("bits", [6, 8])
def test_library_vq_quantizer_is_valid(bits):
    E = 1 << bits
    w = inputs.gen_weight(5, 256, 256, "student")
    blob = B.rwkvq_pack(w, 256, 256, B.RWKVQ_VQ, bits, kmeans_iters=10, seed=7)
    codes = blob.export_codes()
    cb = codes["codebook"][0, 0].astype(np.float64)
    assert np.isfinite(cb).all()
    vecs = w.astype(np.float64).reshape(-1, 2)
    idx = codes["q"].reshape(-1).astype(np.int64)
    d2 = ((vecs[:, None, :] - cb[None, :, :]) ** 2).sum(axis=2)       # brute force, fp64
    assert np.array_equal(d2[np.arange(len(idx)), idx], d2.min(axis=1))  # every index is a nearest centre
    mse_lib = d2.min(axis=1).mean()
    ocb, oix = orc.kmeans_tile(vecs, E, 10, np.random.default_rng(0))
    mse_orc = ((vecs - ocb.astype(np.float64)[oix]) ** 2).sum(axis=1).mean()
    assert mse_lib <= 1.05 * mse_orc


def test_library_vq_zero_error_on_few_distinct_vectors():
    rng = np.random.default_rng(12)
    protos = rng.standard_normal((40, 2)).astype(np.float16)
    w = protos[rng.integers(40, size=256 * 128)].reshape(256, 256)
    blob = B.rwkvq_pack(w, 256, 256, B.RWKVQ_VQ, 6, kmeans_iters=10, seed=1)
    codes = blob.export_codes()
    assert np.array_equal(orc.vq_decode(codes["codebook"], codes["q"]), w.astype(np.float64))


def test_library_mu_quantizer():
    mu = inputs.gen_mu(3, 512)
    blob = B.rwkvq_pack(mu.reshape(1, -1), 1, 512, B.RWKVQ_VQ, 6, seed=2)
    codes = blob.export_codes()
    mh = orc.mu_decode(codes["codebook"], codes["q"])
    assert np.abs(mh - mu.astype(np.float64)).max() < 0.1


def test_error_paths():
    w = inputs.gen_weight(0, 32, 256)
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_pack(w[:, :200], 32, 200, B.RWKVQ_SQ, 3)
    assert e.value.status == 2                                  # ESHAPE
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_pack(w, 32, 256, B.RWKVQ_VQ, 6)                  # VQ matrices need multiples of 256
    assert e.value.status == 2
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_pack(w, 32, 256, B.RWKVQ_SQ, 4)
    assert e.value.status == 7                                  # EUNSUPPORTED
    bad = w.copy()
    bad[1, 1] = np.float16(np.inf)
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_pack(bad, 32, 256, B.RWKVQ_SQ, 3)
    assert e.value.status == 4                                  # ENONFINITE
    q = np.full((32, 256), 9, np.uint8)
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_pack(None, 32, 256, B.RWKVQ_SQ, 3, codes=dict(q=q, scale=np.ones((32, 2), np.float16), zero=np.zeros((32, 2), np.float16)))
    assert e.value.status == 1                                  # EINVAL
    img = B.rwkvq_pack(w, 32, 256, B.RWKVQ_SQ, 3).image()
    with pytest.raises(B.RwkvqError):
        B.rwkvq_image_unpack(img[:1000])                         # truncated
    broken = img.copy()
    broken[0] ^= 0xFF                                            # wrong magic
    with pytest.raises(B.RwkvqError):
        B.rwkvq_image_unpack(broken)
    broken = img.copy()
    broken[300] ^= 0x01                                          # payload bit flip -> CRC mismatch
    with pytest.raises(B.RwkvqError):
        B.rwkvq_image_unpack(broken)
    assert B.lib().rwkvq_status_str(8) == b"device-side wait timed out"


def test_desc_for_matches_the_packer():
    for method, bits, oc, ic in ((B.RWKVQ_SQ, 3, 272, 384), (B.RWKVQ_VQ, 6, 256, 512), (B.RWKVQ_VQ, 8, 512, 256),
                                 (B.RWKVQ_VQ, 6, 1, 514)):
        w = np.zeros((oc, ic), dtype=np.float16)
        blob = B.rwkvq_pack(w, oc, ic, method, bits, kmeans_iters=1)
        d, e = B.rwkvq_desc_for(oc, ic, method, bits), blob.desc
        for f, _ in B.Desc._fields_:
            assert getattr(d, f) == getattr(e, f), f
    with pytest.raises(B.RwkvqError):
        B.rwkvq_desc_for(100, 384, B.RWKVQ_SQ, 3)


def test_tau_for_fraction_matches_oracle():
    from oracle import rwkvq_oracle as orc
    rng = np.random.default_rng(8)
    for m in (1, 2, 7, 40):
        vals = rng.standard_normal(m) * 3.0
        for frac in (0.0, 0.1, 0.5, 0.9, 1.0):
            a, b = B.rwkvq_tau_for_fraction(vals, frac), orc.tau_for_fraction(vals, frac)
            assert a == b or (np.isinf(a) and np.isinf(b) and a * b > 0)
    with pytest.raises(B.RwkvqError):
        B.rwkvq_tau_for_fraction([1.0, float("nan")], 0.5)
    with pytest.raises(B.RwkvqError):
        B.rwkvq_tau_for_fraction([1.0], 1.5)


def test_tau_largest_gap_separates_two_clusters():
    """Worked cases: the threshold is the midpoint of the widest gap of the sorted finite values."""
    assert B.rwkvq_tau_largest_gap([1.0, 1.2, 5.0, 1.1, 5.5]) == 0.5 * (1.2 + 5.0)
    assert B.rwkvq_tau_largest_gap([3.0, 1.0, 2.0]) == 1.5              # equal gaps: the first one
    assert B.rwkvq_tau_largest_gap([0.25, float("inf"), 0.75]) == 0.5    # non-finite values are ignored
    assert np.isinf(B.rwkvq_tau_largest_gap([2.0, 2.0, 2.0])) and B.rwkvq_tau_largest_gap([2.0, 2.0]) > 0
    assert np.isinf(B.rwkvq_tau_largest_gap([7.0]))
    rng = np.random.default_rng(3)
    lo, hi = rng.uniform(0.0, 1.0, 40), rng.uniform(3.0, 4.0, 6)
    tau = B.rwkvq_tau_largest_gap(rng.permutation(np.concatenate([lo, hi])))
    assert tau == 0.5 * (lo.max() + hi.min())
    with pytest.raises(B.RwkvqError):
        B.rwkvq_tau_largest_gap([1.0, float("nan")])
