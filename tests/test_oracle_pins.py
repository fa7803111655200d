"""Pins for the CPU oracle: closed forms, hand-worked values, invariants and
brute force on tiny inputs.  None of these tests touches the CUDA library."""
import math
import os

import numpy as np
import pytest

from oracle import rwkvq_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(t) for t in line.split()])
    return rows


# ---------------------------------------------------------------- SQ (Eq. 2)

def test_sq_identity_8bit_unit_scale():
    # 8-bit codes with s = 1, z = 0 decode to themselves
    q = np.arange(256, dtype=np.uint8).reshape(2, 128)
    s = np.ones((2, 1), np.float16)
    z = np.zeros((2, 1), np.float16)
    assert np.array_equal(orc.sq_decode(q, s, z), np.arange(256, dtype=np.float64).reshape(2, 128))


def test_sq_decode_every_code_and_zero_point():
    # s*(q-z) for every (q, z) in [0,7]^2 and several fp16 scales, against integer arithmetic
    for s_val in (0.5, 0.0173, 3.0, 2.0 ** -14):
        s16 = np.float16(s_val)
        for zz in range(8):
            q = np.tile(np.arange(8, dtype=np.uint8), 16)[None, :]
            out = orc.sq_decode(q, np.array([[s16]]), np.array([[np.float16(zz)]]))
            for j in range(128):
                assert out[0, j] == float(s16) * (int(q[0, j]) - zz)


def test_sq_encode_ramp_and_shifted_ramp():
    ramp = np.tile(np.arange(8), 16).astype(np.float16)[None, :]  # min 0, max 7 -> s=1, z=0, q=w
    q, s, z = orc.sq_encode(ramp)
    assert float(s[0, 0]) == 1.0 and float(z[0, 0]) == 0.0 and np.array_equal(q, ramp.astype(np.uint8))
    shifted = (ramp.astype(np.float64) * 0.5 - 1.0).astype(np.float16)  # min -1, s=.5 -> z = 2
    q, s, z = orc.sq_encode(shifted)
    assert float(s[0, 0]) == 0.5 and float(z[0, 0]) == 2.0
    assert np.array_equal(q, ramp.astype(np.uint8))
    assert np.array_equal(orc.sq_decode(q, s, z), shifted.astype(np.float64))


def test_sq_encode_groups_run_along_input_dim():
    # two groups in one row with different ranges must get different scales;
    # two rows must not share a group
    w = np.zeros((2, 256), np.float16)
    w[0, :128] = np.tile(np.arange(8), 16)
    w[0, 128:] = np.tile(np.arange(8), 16) * 2
    w[1, :128] = np.tile(np.arange(8), 16) * 4
    w[1, 128:] = np.tile(np.arange(8), 16) * 8
    q, s, z = orc.sq_encode(w)
    assert s.shape == (2, 2)
    assert [float(v) for v in s.reshape(-1)] == [1.0, 2.0, 4.0, 8.0]
    assert np.array_equal(orc.sq_decode(q, s, z), w.astype(np.float64))


def test_sq_reconstruction_error_bound():
    rng = np.random.default_rng(1)
    w = (rng.standard_normal((8, 512)) * 0.02).astype(np.float16)
    q, s, z = orc.sq_encode(w)
    assert q.max() <= 7 and q.min() >= 0
    zz = z.astype(np.float64)
    assert np.array_equal(zz, np.rint(zz)) and zz.min() >= 0 and zz.max() <= 7
    err = np.abs(orc.sq_decode(q, s, z) - w.astype(np.float64)).reshape(8, 4, 128)
    sg = s.astype(np.float64)[:, :, None]
    inner = (q.reshape(8, 4, 128) > 0) & (q.reshape(8, 4, 128) < 7)
    assert (err[inner] <= (0.5 * sg * (1 + 1e-12) + 0 * err)[inner]).all()
    assert (err <= 1.5 * sg).all()
    # every code is used somewhere (a dropped zero point or a wrong sign collapses the range)
    assert set(np.unique(q)) == set(range(8))


def test_sq_degenerate_groups():
    for c, exp in ((0.0, (1.0, 0.0, 0)), (0.25, (0.25, 0.0, 1)), (-0.75, (0.75, 1.0, 0))):
        w = np.full((1, 128), c, np.float16)
        q, s, z = orc.sq_encode(w)
        assert (float(s[0, 0]), float(z[0, 0]), int(q[0, 0])) == exp
        assert np.array_equal(orc.sq_decode(q, s, z), w.astype(np.float64))
    # scale underflow (range below 7 * 2^-25) is coded as the constant min
    w = np.zeros((1, 128), np.float16)
    w[0, 5] = np.float16(2.0 ** -24)
    q, s, z = orc.sq_encode(w)
    assert np.array_equal(orc.sq_decode(q, s, z), np.zeros((1, 128)))


def test_bpw_arithmetic_matches_paper_operating_point():
    sq_bpw, vq_bpw, f_sq, f_vq, avg = _gold("bpw.txt")[0]
    assert 3 + (16 + 16) / 128 == sq_bpw           # 3-bit codes + fp16 s and z per 128 weights
    assert abs(f_sq * sq_bpw + f_vq * vq_bpw - avg) < 1e-12
    assert 6 / 2 + 64 * 2 * 16 / (256 * 256) == 3.03125   # this build's VQ: 6-bit index per 2 weights + codebook


# ---------------------------------------------------------------- VQ (Eq. 3)

def test_vq_one_entry_codebook_is_constant_matrix():
    cbs = np.zeros((1, 1, 1, 2), np.float16)
    cbs[0, 0, 0] = (0.125, -0.5)
    idx = np.zeros((256, 128), np.uint8)
    out = orc.vq_decode(cbs, idx)
    assert (out[:, 0::2] == 0.125).all() and (out[:, 1::2] == -0.5).all()


def test_vq_decode_counter_pattern_and_tile_grid():
    # 2 x 3 tile grid with distinct codebooks: entry e of tile (i,j) = (100 i + 10 j + e/64, -that)
    tile, E = 256, 64
    cbs = np.zeros((2, 3, E, 2), np.float16)
    for i in range(2):
        for j in range(3):
            for e in range(E):
                v = np.float16(4 * i + j + e / 64.0)
                cbs[i, j, e] = (v, -v)
    idx = (np.arange(512 * 384).reshape(512, 384) % E).astype(np.uint8)
    out = orc.vq_decode(cbs, idx)
    for (r, c) in ((0, 0), (300, 2), (511, 767), (255, 256), (256, 255), (17, 513)):
        i, j, p = r // tile, c // tile, c // 2
        e = (r * 384 + p) % E
        v = float(np.float16(4 * i + j + e / 64.0))
        assert out[r, c] == (v if c % 2 == 0 else -v)


def test_vq_vectors_are_row_major_pairs():
    # rows alternate (1,2,1,2,...) / (3,4,3,4,...): exactly two distinct row-major pairs
    w = np.zeros((256, 256), np.float16)
    w[0::2, 0::2], w[0::2, 1::2] = 1, 2
    w[1::2, 0::2], w[1::2, 1::2] = 3, 4
    cbs, idx = orc.vq_encode(w, entries=2, iters=3, seed=3)
    assert np.array_equal(orc.vq_decode(cbs, idx), w.astype(np.float64))
    got = {tuple(float(v) for v in cbs[0, 0, e]) for e in range(2)}
    assert got == {(1.0, 2.0), (3.0, 4.0)}


def test_kmeans_zero_error_when_distinct_vectors_fit_codebook():
    rng = np.random.default_rng(5)
    protos = rng.standard_normal((16, 2)).astype(np.float16).astype(np.float64)
    protos = np.unique(protos, axis=0)
    vecs = protos[rng.integers(len(protos), size=4000)]
    cb, ix = orc.kmeans_tile(vecs, len(protos), 10, np.random.default_rng(0))
    assert np.array_equal(cb.astype(np.float64)[ix], vecs)


def test_kmeans_lloyd_loss_monotone_and_assignment_is_nearest():
    rng = np.random.default_rng(6)
    vecs = (rng.standard_normal((600, 2)) * 0.02).astype(np.float16).astype(np.float64)
    cb, ix, losses = orc.kmeans_tile(vecs, 8, 10, np.random.default_rng(1), return_losses=True)
    body = losses[:-1]
    assert all(b <= a * (1 + 1e-12) for a, b in zip(body, body[1:]))
    assert body[-1] < body[0]
    c = cb.astype(np.float64)
    for i in range(len(vecs)):  # brute force, ties to the lowest index
        d = [(vecs[i, 0] - c[e, 0]) ** 2 + (vecs[i, 1] - c[e, 1]) ** 2 for e in range(8)]
        assert ix[i] == d.index(min(d))


def test_weighted_kmeans_minimises_weighted_loss():
    # Section 4.2: with weights X^2 the centre of a cluster is the weighted mean.
    vecs = np.array([[0.0, 0.0], [1.0, 1.0]] * 8)
    wts = np.array([[1.0, 1.0], [3.0, 3.0]] * 8)
    cb, ix = orc.kmeans_tile(vecs, 1, 3, np.random.default_rng(0), weights=wts)
    assert np.allclose(cb.astype(np.float64)[0], [0.75, 0.75])


def test_weighted_kmeans_both_half_steps_lower_eq19():
    # Eq. 19: with element weights X^2 spanning six decades, assignment by weighted distance and
    # weighted means never raise the loss; the final assignment is the brute-force weighted argmin.
    rng = np.random.default_rng(11)
    vecs = rng.uniform(0.0, 1.0, (400, 2)).astype(np.float16).astype(np.float64)
    wts = 10.0 ** rng.uniform(-3.0, 3.0, (400, 2))
    cb, ix, losses = orc.kmeans_tile(vecs, 8, 10, np.random.default_rng(2), weights=wts, return_losses=True)
    body = losses[:-1]
    assert all(b <= a * (1 + 1e-12) for a, b in zip(body, body[1:]))
    assert body[-1] < body[0]
    c = cb.astype(np.float64)
    for i in range(len(vecs)):
        d = [wts[i, 0] * (vecs[i, 0] - c[e, 0]) ** 2 + wts[i, 1] * (vecs[i, 1] - c[e, 1]) ** 2 for e in range(8)]
        assert ix[i] == d.index(min(d))
    # an unweighted assignment is a different (worse or equal) answer under Eq. 19
    ix_plain = orc._nearest(vecs, c)
    loss_w = float((wts * (vecs - c[ix]) ** 2).sum())
    loss_p = float((wts * (vecs - c[ix_plain]) ** 2).sum())
    assert loss_w <= loss_p and not np.array_equal(ix, ix_plain)


def test_weighted_kmeans_zero_weight_elements_do_not_move_centres():
    # vectors whose weights are zero contribute nothing to Eq. 19: the single centre sits on the
    # weighted members' mean however far the unweighted ones are.
    vecs = np.array([[0.25, 0.5]] * 4 + [[100.0, -100.0]] * 4)
    wts = np.array([[2.0, 2.0]] * 4 + [[0.0, 0.0]] * 4)
    cb, _ = orc.kmeans_tile(vecs, 1, 2, np.random.default_rng(0), weights=wts)
    assert np.array_equal(cb.astype(np.float64)[0], [0.25, 0.5])


def test_representative_activation_hand_worked():
    # Section 4.2.  Four samples 0, 1, 2, 10 of one position, pct = 25: the percentiles by linear
    # interpolation sit at positions 0.75 and 2.25 of the sorted samples, i.e. 0.75 and
    # 2 + 0.25 * 8 = 4; the limited samples 0.75, 1, 2, 4 average to 1.9375 (plain mean 3.25).
    x = np.array([[2.0], [10.0], [0.0], [1.0]])
    assert orc.representative_activation(x, 25.0)[0] == 1.9375
    assert orc.representative_activation(x, 0.0)[0] == 3.25
    # 101 samples 0..99 and one outlier 10000, pct = 10: limits are the order statistics 10 and
    # 90, the limited samples sum to 10*10 + (10+...+90) + 10*90 = 5050, mean 50 (plain mean 148.02).
    col = np.concatenate([np.arange(100.0), [10000.0]])
    rep = orc.representative_activation(np.random.default_rng(0).permutation(col)[:, None], 10.0)
    assert abs(rep[0] - 50.0) < 1e-12
    assert abs(orc.representative_activation(col[:, None], 0.0)[0] - 14950.0 / 101.0) < 1e-12


def test_representative_activation_matches_winsorised_mean_on_order_statistics():
    # Where the percentiles fall exactly on order statistics the clipped mean is the winsorised
    # mean of a statistics library.
    from scipy.stats.mstats import winsorize
    rng = np.random.default_rng(4)
    x = rng.standard_normal((101, 7))
    x[rng.integers(0, 101, 5), rng.integers(0, 7, 5)] *= 50.0
    rep = orc.representative_activation(x, 10.0)
    for j in range(7):
        ref = float(np.asarray(winsorize(x[:, j], limits=(0.1, 0.1))).mean())
        assert abs(rep[j] - ref) < 1e-12
    # constant positions stay put; each position is treated on its own
    y = np.tile(np.array([[1.5, -2.0]]), (9, 1))
    assert np.array_equal(orc.representative_activation(y, 5.0), [1.5, -2.0])


def test_mu_roundtrip_shapes():
    mu = np.linspace(0.0, 1.0, 512).astype(np.float16)
    cb, ix = orc.mu_encode(mu, entries=64, iters=10, seed=0)
    assert cb.shape == (64, 2) and ix.shape == (256,)
    mh = orc.mu_decode(cb, ix)
    assert mh.shape == (512,) and np.abs(mh - mu.astype(np.float64)).max() < 0.02


def test_mu_encode_reproduces_few_distinct_pairs_in_order():
    # A vector made of no more distinct (even, odd) pairs than codebook entries is coded without
    # error, and decoding puts every pair back at its own position: a reshape that paired the wrong
    # elements (stride ic/2 instead of 2, or columns swapped) would either need more than `entries`
    # centres or return the halves in the wrong order.
    rng = np.random.default_rng(5)
    pairs = (rng.random((48, 2)) * 0.9 + 0.05).astype(np.float16)
    pairs[:, 1] += np.float16(1.0)                       # odd elements in (1, 2), even ones in (0, 1)
    which = rng.integers(0, 48, size=300)
    mu = pairs[which].reshape(-1)                        # [x0, y0, x1, y1, ...]
    cb, ix = orc.mu_encode(mu, entries=64, iters=10, seed=3)
    mh = orc.mu_decode(cb, ix)
    assert np.array_equal(mh, mu.astype(np.float64))
    assert (mh[0::2] < 1.0).all() and (mh[1::2] >= 1.0).all()
    # the indices name the pair each position holds: equal pairs share an index, different pairs do not
    for a, b in [(0, 1), (5, 200), (17, 299)]:
        assert (ix[a] == ix[b]) == bool((pairs[which[a]] == pairs[which[b]]).all())


# ---------------------------------------------------------------- proxy (Eqs. 5-18)

def test_proxy_hand_worked_three_elements():
    pc_g, pf2_g, pf4_g = _gold("proxy_hand.txt")[0]
    pc, pf4 = orc.proxy(np.array([[3.0, 0.0, 1.0]]), K=4)
    _, pf2 = orc.proxy(np.array([[3.0, 0.0, 1.0]]), K=2)
    assert abs(pc - pc_g) < 1e-13 and abs(pf2 - pf2_g) < 1e-13 and abs(pf4 - pf4_g) < 1e-13


def test_proxy_family_hand_worked_and_closed_forms():
    # Three weights 3, 0, 1: sorted 0, 1, 3, gaps 1, 2, G' = 1/3, 2/3, n = 2, mean 1/2.  By hand:
    # variance = ((1/6)^2 + (1/6)^2) / 2 = 1/36, cv = (1/6) / (1/2) = 1/3, range = 1/3, mad = 1/6,
    # ie = -(1/3 ln 1/3 + 2/3 ln 2/3) = ln 3 - (2/3) ln 2.
    f = orc.proxy_family(np.array([[3.0, 0.0, 1.0]]))
    assert abs(f["variance"] - 1.0 / 36.0) < 1e-15 and abs(f["cv"] - 1.0 / 3.0) < 1e-15
    assert abs(f["range"] - 1.0 / 3.0) < 1e-15 and abs(f["mad"] - 1.0 / 6.0) < 1e-15
    assert abs(f["ie"] - (np.log(3.0) - 2.0 / 3.0 * np.log(2.0))) < 1e-15
    # equispaced weights: every gap equal, so every dispersion statistic is 0 and ie = ln n
    w = np.random.default_rng(0).permutation(np.arange(4096) * 0.125 - 7.0).reshape(64, 64)
    f = orc.proxy_family(w)
    assert max(f["variance"], f["cv"], f["range"], f["mad"]) < 1e-12 and abs(f["ie"] - np.log(4095.0)) < 1e-9
    # m + 1 levels each repeated r times: m gaps of 1/m, n - m ties, n = (m + 1) r - 1
    m, r = 7, 5
    w = np.repeat(np.arange(m + 1.0), r)
    n = (m + 1) * r - 1
    f = orc.proxy_family(w.reshape(1, -1))
    var = (m * (1.0 / m - 1.0 / n) ** 2 + (n - m) * (1.0 / n) ** 2) / n
    assert abs(f["variance"] - var) < 1e-15 and abs(f["cv"] - np.sqrt(var) * n) < 1e-12
    assert abs(f["range"] - 1.0 / m) < 1e-15 and abs(f["ie"] - np.log(m)) < 1e-14
    assert abs(f["mad"] - (m * (1.0 / m - 1.0 / n) + (n - m) / n) / n) < 1e-15
    # ties to the coarse proxy and to the second moment of the fine proxy
    w = (np.random.default_rng(3).standard_normal((32, 48)) * 0.02).astype(np.float16)
    f = orc.proxy_family(w)
    pc, pf2 = orc.proxy(w, K=2)
    nn = w.size - 1
    assert abs((np.log(nn) - f["ie"]) - pc) < 1e-12 and abs(f["variance"] * nn ** 2 / 2.0 - pf2) < 1e-9 * pf2
    assert all(np.isinf(v) for v in orc.proxy_family(np.full((4, 4), 0.5)).values())


def test_quant_sse_closed_forms():
    assert orc.quant_sse(np.array([[0.0, 1.0], [2.0, 3.0]]), np.array([[0.0, 1.0], [2.0, 5.0]])) == 4.0
    # uniform quantization of a dense ramp with step s: errors are k*s/m - round, sum known
    w16 = (np.arange(128) % 8 * 0.125).astype(np.float16).reshape(1, 128)      # exactly representable levels
    q, s_, z = orc.sq_encode(w16)
    assert orc.quant_sse(w16, orc.sq_decode(q, s_, z)) == 0.0
    # two values around one level: errors +-d each
    assert abs(orc.quant_sse(np.array([0.25, 0.75]), np.array([0.5, 0.5])) - 0.125) < 1e-16


def test_tau_for_fraction_sends_the_stated_share_to_sq():
    vals = np.random.default_rng(5).permutation(np.arange(20) * 1.5 + 0.25)
    for frac, k in ((0.9, 18), (0.5, 10), (0.0, 0), (1.0, 20), (0.33, 7)):
        tau = orc.tau_for_fraction(vals, frac)
        assert int((vals < tau).sum()) == k
    assert orc.tau_for_fraction([1.0, 2.0, 4.0, 8.0], 0.5) == 3.0


def test_proxy_equispaced_is_zero():
    w = (np.arange(4096, dtype=np.float64) * 0.125 - 7.0).reshape(64, 64)
    rng = np.random.default_rng(0)
    pc, pf = orc.proxy(rng.permutation(w.reshape(-1)).reshape(64, 64), K=6)
    assert abs(pc) < 1e-9 and abs(pf) < 1e-9


def test_proxy_two_level_closed_form_with_ties():
    # values 0..m each repeated r times: m gaps of 1/m, the other n-m gaps are ties (zero)
    m, r = 7, 9
    w = np.repeat(np.arange(m + 1, dtype=np.float64), r)
    n = w.size - 1
    pc, pf = orc.proxy(w.reshape(8, 9), K=4)
    assert abs(pc - (math.log(n) - math.log(m))) < 1e-12
    exp = 0.0
    for k in (2, 3, 4):
        mk = (m * (1.0 / m - 1.0 / n) ** k + (n - m) * (-1.0 / n) ** k) / n
        exp += n ** k / (k * (k - 1)) * abs(mk)
    assert abs(pf - exp) < 1e-9 * exp


def test_proxy_bruteforce_tiny_with_ties():
    rng = np.random.default_rng(11)
    for trial in range(6):
        w = rng.integers(-5, 6, size=(4, 8)).astype(np.float64) * 0.25
        vals = sorted(float(v) for v in w.reshape(-1))
        gaps = [vals[i + 1] - vals[i] for i in range(len(vals) - 1)]
        n = len(gaps)
        tot = sum(gaps)
        gp = [g / tot for g in gaps]
        h = -sum(p * math.log(p) for p in gp if p > 0)
        pc_ref = math.log(n) - h
        pf_ref = 0.0
        for k in range(2, 5):
            mk = sum((p - 1.0 / n) ** k for p in gp) / n
            pf_ref += n ** k / (k * (k - 1)) * abs(mk)
        assert abs(sum(p - 1.0 / n for p in gp)) < 1e-12     # Eq. 11
        pc, pf = orc.proxy(w, K=4)
        assert abs(pc - pc_ref) < 1e-12 and abs(pf - pf_ref) < 1e-9 * max(1.0, pf_ref)


def test_proxy_invariants():
    rng = np.random.default_rng(2)
    w = rng.standard_normal((32, 64))
    pc, pf = orc.proxy(w)
    assert pc >= 0.0
    pc2, pf2 = orc.proxy(3.5 * w.T.copy() - 2.0)       # affine map and reshape leave G' unchanged
    assert abs(pc - pc2) < 1e-9 and abs(pf - pf2) < 1e-6 * pf
    assert orc.proxy(np.full((4, 4), 0.5)) == (math.inf, math.inf)


def test_proxy_taylor_sum_matches_pc_near_uniform():
    rng = np.random.default_rng(3)
    gaps = 1.0 + 0.05 * rng.standard_normal(100_000)
    w = np.concatenate([[0.0], np.cumsum(gaps)])
    pc, _ = orc.proxy(w.reshape(1, -1))
    signed = orc.proxy_taylor_signed(w.reshape(1, -1), K=6)
    assert pc > 1e-3 and abs(signed - pc) < 1e-3 * pc
    # and P_f >= |signed sum| because it adds magnitudes (Eq. 17 vs Eq. 15)
    _, pf = orc.proxy(w.reshape(1, -1), K=6)
    assert pf >= abs(signed) * (1 - 1e-12)


def test_proxy_iid_uniform_limit():
    # normalised spacings of an iid uniform sample are ~Exp(1)/n: P_c -> 1 - Euler gamma
    rng = np.random.default_rng(4)
    pc, pf = orc.proxy(rng.random((512, 512)))
    assert abs(pc - (1 - 0.5772156649)) < 0.01
    # E[(t-1)^k], t~Exp(1): 1, 2, 9  ->  P_f(K=4) -> 1/2 + 2/6 + 9/12
    assert abs(pf - (0.5 + 2 / 6 + 9 / 12)) < 0.1


def test_selection_rule_three_branches():
    rows = _gold("thresholds.txt")
    tau_c, tau_f = rows[1]
    rng = np.random.default_rng(7)
    uniform = rng.random((128, 128))
    outl = uniform.copy()
    outl[0, :2] = [1.01, -0.008]      # two values just outside the bulk: two wide gaps
    heavy = rng.standard_t(2.0, size=(128, 128))
    (pc_u, pf_u), (pc_o, pf_o), (pc_h, pf_h) = orc.proxy(uniform), orc.proxy(outl), orc.proxy(heavy)
    assert pc_u < tau_c and pf_u < tau_f and orc.select(pc_u, pf_u, tau_c, tau_f) == 1
    assert pc_o < tau_c and pf_o >= tau_f and orc.select(pc_o, pf_o, tau_c, tau_f) == 0
    assert pc_h >= tau_c and orc.select(pc_h, pf_h, tau_c, tau_f) == 0
    # strictness (Eq. 18): equality goes to VQ
    assert orc.select(tau_c, 0.0, tau_c, tau_f) == 0 and orc.select(0.0, tau_f, tau_c, tau_f) == 0
    assert orc.select(math.inf, math.inf, tau_c, tau_f) == 0


# ---------------------------------------------------------------- runtime math

def test_token_shift_special_cases():
    x = np.array([[1.0, 2.0, 3.0, 4.0]])
    xp = np.array([[10.0, 20.0, 30.0, 40.0]])
    assert np.array_equal(orc.token_shift(x, xp, np.zeros(4)), x)
    assert np.array_equal(orc.token_shift(x, xp, np.ones(4)), xp)
    assert np.array_equal(orc.token_shift(x, xp, np.array([0.5, 0.0, 1.0, 0.25])),
                          np.array([[5.5, 2.0, 30.0, 13.0]]))
    # same interpolation as mu_p*x + (1-mu_p)*x_prev with mu_p = 1 - mu_hat (Eq. 20)
    mu_hat = np.array([0.125, 0.5, 0.75, 1.0])
    assert np.allclose(orc.token_shift(x, xp, mu_hat), (1 - mu_hat) * x + mu_hat * xp, rtol=0, atol=1e-15)


def test_gemv_against_loops_and_identity():
    rng = np.random.default_rng(8)
    w = rng.standard_normal((5, 7))
    x = rng.standard_normal((3, 7))
    y = orc.gemv(w, x)
    assert y.shape == (3, 5)
    for b in range(3):
        for i in range(5):
            assert abs(y[b, i] - sum(w[i, j] * x[b, j] for j in range(7))) < 1e-13
    assert np.array_equal(orc.gemv(np.eye(7), x), x)
    # row/column roles: a matrix with a single one at [i=2, j=4] copies x[:,4] into y[:,2]
    e = np.zeros((5, 7))
    e[2, 4] = 1.0
    yy = orc.gemv(e, x)
    assert np.array_equal(yy[:, 2], x[:, 4]) and np.count_nonzero(yy) == 3


def test_tolerance_formula():
    w = np.array([[3.0, 4.0], [0.0, 1.0]])
    x = np.array([[6.0, 8.0]])
    assert np.allclose(orc.tolerance(w, x), [[2e-3 * 5 * 10, 2e-3 * 1 * 10]])


def test_prefill_prev_rows():
    X = np.arange(12, dtype=np.float64).reshape(4, 3)
    P = orc.prefill_prev(X, None)
    assert np.array_equal(P[0], np.zeros(3)) and np.array_equal(P[1:], X[:-1])
    P = orc.prefill_prev(X, np.array([7.0, 8.0, 9.0]))
    assert np.array_equal(P[0], [7.0, 8.0, 9.0])


def test_bf16_rounding_ties_to_even():
    vals = np.array([1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -3.0])
    out = orc.bf16_rne(vals)
    assert [float(v) for v in out] == [1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -3.0]


def test_proxy_segments_closed_forms_per_tile():
    """Per-tile proxy: a tile that is an equispaced ramp (in any order) has P_c = P_f = 0 exactly up to
    rounding, a tile of two clusters has P_c > 0, a constant tile and a one-element tile give inf; the tile
    grid is ragged at the edges."""
    rng = np.random.default_rng(5)
    w = np.zeros((5, 7))
    w[0:2, 0:3] = rng.permutation(np.arange(6.0)).reshape(2, 3) * 0.25 - 1.0      # ramp
    w[0:2, 3:6] = np.array([[0.0, 0.001, 0.002], [5.0, 5.001, 5.002]])            # two clusters
    w[0:2, 6:7] = np.array([[1.0], [3.0]])                                        # two elements: one gap, g' = 1
    w[2:4, 0:3] = 2.5                                                             # constant
    w[2:4, 3:6] = rng.standard_normal((2, 3))
    w[4:5, 6:7] = 9.0                                                             # single element
    pc, pf = orc.proxy_segments(w, 2, 3, K=4)
    assert pc.shape == (3, 3)
    assert abs(pc[0, 0]) < 1e-12 and abs(pf[0, 0]) < 1e-12
    assert pc[0, 1] > 0.5 and pf[0, 1] > 0.0
    # n = 1: P_c = ln 1 - 0 = 0 and delta = 0
    assert pc[0, 2] == 0.0 and pf[0, 2] == 0.0
    assert np.isinf(pc[1, 0]) and np.isinf(pf[1, 0])
    assert np.isinf(pc[2, 2]) and np.isinf(pf[2, 2])
    a, b = orc.proxy(w[2:4, 3:6], 4)
    assert pc[1, 1] == a and pf[1, 1] == b
    # whole matrix as one tile = the matrix-level proxy
    pcm, pfm = orc.proxy_segments(w, 5, 7, K=4)
    assert (pcm[0, 0], pfm[0, 0]) == orc.proxy(w, 4)


def test_wkv_recurrence_equals_the_literal_sums_and_closed_forms():
    """Eq. 23: the two-sum recurrence reproduces the written-out sums token by token; first token gives v;
    with no decay and no bonus the result is the softmax(k)-weighted mean of v; a huge decay keeps the previous and the current token only."""
    rng = np.random.default_rng(9)
    T, d = 7, 5
    ks, vs = rng.standard_normal((T, d)), rng.standard_normal((T, d))
    u, w = rng.standard_normal(d) * 0.5, rng.uniform(0.1, 1.5, d)
    a, b = np.zeros(d), np.zeros(d)
    for t in range(1, T + 1):
        wkv, a, b = orc.wkv_step(a, b, ks[t - 1], vs[t - 1], u, w)
        ref = orc.wkv_literal(ks[:t], vs[:t], u, w)
        assert np.allclose(wkv, ref, rtol=1e-12, atol=1e-14)
        if t == 1:
            assert np.allclose(wkv, vs[0], rtol=1e-14)
    # w = 0, u = 0: every token weighs exp(k_i) -> softmax-weighted mean over the history
    z = np.zeros(d)
    got = orc.wkv_literal(ks, vs, z, z)
    p = np.exp(ks) / np.exp(ks).sum(axis=0)
    assert np.allclose(got, (p * vs).sum(axis=0), rtol=1e-12)
    # very large decay: f(i) keeps only i = t - 1 (its exponent carries no multiple of w), so the result
    # mixes the previous and the current token with weights e^{k_{t-1}} and e^{u + k_t}
    e_prev, e_cur = np.exp(ks[-2]), np.exp(u + ks[-1])
    assert np.allclose(orc.wkv_literal(ks, vs, u, np.full(d, 700.0)), (e_prev * vs[-2] + e_cur * vs[-1]) / (e_prev + e_cur),
                       rtol=1e-12)
    # hand-worked: one channel, two tokens, k = 0, u = 0, w = ln 2: wkv_2 = (v1 + v2) / 2 ... f(1) = exp(0) = 1
    one = orc.wkv_literal(np.zeros((2, 1)), np.array([[2.0], [6.0]]), np.zeros(1), np.array([math.log(2.0)]))
    assert np.allclose(one, [4.0])
    # three tokens: f(1) = exp(-w) = 1/2, f(2) = 1: (0.5*2 + 1*6 + 1*10) / (0.5 + 1 + 1)
    three = orc.wkv_literal(np.zeros((3, 1)), np.array([[2.0], [6.0], [10.0]]), np.zeros(1), np.array([math.log(2.0)]))
    assert np.allclose(three, [17.0 / 2.5])


def test_gates_closed_forms():
    assert orc.sigmoid(np.array([0.0]))[0] == 0.5
    x = np.array([-3.0, 0.5, 2.0])
    assert np.allclose(orc.sigmoid(x) + orc.sigmoid(-x), 1.0)
    assert np.array_equal(orc.relu_squared(np.array([-2.0, 0.0, 3.0])), np.array([0.0, 0.0, 9.0]))
    assert np.allclose(orc.time_mix_gate(np.zeros(3), x), 0.5 * x)
    assert np.allclose(orc.channel_mix_gate(np.full(3, 50.0), x), x)


def test_rms_normalize_closed_forms():
    x = np.array([[3.0, -3.0, 3.0, -3.0], [0.5, 0.0, 0.0, 0.0]])
    y = orc.rms_normalize(x, eps=0.0)
    assert np.allclose(y[0], [1.0, -1.0, 1.0, -1.0]) and np.allclose(y[1], [2.0, 0.0, 0.0, 0.0])
    z = np.random.default_rng(2).standard_normal((3, 64))
    n = orc.rms_normalize(z, eps=0.0)
    assert np.allclose((n * n).mean(axis=1), 1.0) and np.allclose(orc.rms_normalize(7.5 * z, eps=0.0), n)
    assert np.array_equal(orc.rms_normalize(np.zeros((1, 8))), np.zeros((1, 8)))      # eps keeps a zero row finite
