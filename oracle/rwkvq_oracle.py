"""CPU oracle for the hybrid scalar/vector-quantized RWKV projection path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA
library is checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product never does, and this
file imports nothing from the product except nothing at all (numpy only).

All floating-point work is float64 on values that are exactly representable
(fp16 weights, fp16 scales / zero points / codebook entries, fp16 or bf16
activations), so every decoded weight below is the exact real number the
format denotes.

Passages followed (RWKVQuant, arXiv 2505.03803):
  * scalar quantizer                     -- Section 3.2, Eq. 2  (uniform b-bit, scale/zero point)
  * vector quantizer                     -- Section 3.2, Eq. 3  (nearest codebook row, (2^k, d) codebook)
  * codebook by k-means                  -- Section 3.2 (K-Means clustering of source vectors)
  * coarse proxy P_c                     -- Section 4.1, Eqs. 5-9
  * fine proxy P_f                       -- Section 4.1, Eqs. 10-17
  * selection rule phi                   -- Section 4.1, Eq. 18
  * other statistics of G' (ablation)    -- Section 5.3 (Variance, CV, Range, MAD, IE); thresholds for a
                                            target SQ share -- Section 5.1
  * token shift mix and projections      -- Appendix A.1, Eqs. 20-22, 24-27
  * WKV, sigmoid gates, squared ReLU     -- Appendix A.1, Eq. 23 (wkv), Eq. 24 (sigma(r) * wkv),
                                            Eq. 27 (sigma(r') * (W'_v . max(k', 0)^2))
  * weighted loss for element-wise mu    -- Section 4.2, Eq. 19 (weighted k-means; representative X by
                                            percentile clipping before the mean)

Pin status: every function here is pinned by tests/test_oracle_pins.py to
closed forms, invariants or brute force, except `vq_kmeans` codebook *values*
(several correct results exist; parity unpinned by design -- validity
properties are pinned instead: zero error on <=E distinct vectors,
monotone Lloyd loss, nearest-centre assignment).
"""
from __future__ import annotations

import math

import numpy as np

# --------------------------------------------------------------------------
# number-format helpers (no method arithmetic)
# --------------------------------------------------------------------------


def f16(a) -> np.ndarray:
    """Round to IEEE binary16 (nearest even), as numpy float16."""
    return np.asarray(a, dtype=np.float64).astype(np.float16)


def bf16_rne(a) -> np.ndarray:
    """Round float64/float32 values that are exactly representable in float32 to
    bfloat16 (nearest even); returns float32 holding the bf16 values."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    assert np.array_equal(f.astype(np.float64), np.asarray(a, dtype=np.float64)), "input not fp32-exact"
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    out = (((u + r) >> 16) << 16).astype(np.uint32)
    return out.view(np.float32).reshape(f.shape)


# --------------------------------------------------------------------------
# Scalar quantization, Section 3.2 Eq. 2
# --------------------------------------------------------------------------


def sq_encode(w16: np.ndarray, bits: int = 3, group: int = 128):
    """Round-to-nearest group-wise asymmetric uniform quantizer.

    Per group of `group` consecutive input-dim weights of one row (Eq. 2):
        s = (max - min) / (2^b - 1)          (the printed "/2^b-1" read as one denominator)
        z = round(-min / s)                  (integer zero point, clamped to the code range)
        q = clamp(round(w / s) + z, 0, 2^b - 1)
    s is stored as fp16 and the *stored* s is the one used for z and q; rounding
    is to nearest with ties to even.  Degenerate groups (max == min, or a scale
    that underflows to 0 in fp16) are coded as a constant c = min:
        c == 0 -> (s, z, q) = (1, 0, 0);  c > 0 -> (c, 0, 1);  c < 0 -> (|c|, 1, 0).

    Returns q uint8 [oc, ic], s float16 [oc, ic/group], z float16 [oc, ic/group].
    """
    w = np.asarray(w16, dtype=np.float16)
    oc, ic = w.shape
    assert ic % group == 0
    qmax = (1 << bits) - 1
    wg = w.astype(np.float64).reshape(oc, ic // group, group)
    mn = wg.min(axis=2)
    mx = wg.max(axis=2)
    s = ((mx - mn) / qmax).astype(np.float16)  # single RNE rounding from float64
    s64 = s.astype(np.float64)
    degenerate = (mx == mn) | (s64 == 0.0)
    safe = np.where(degenerate, 1.0, s64)
    z = np.clip(np.rint(-mn / safe), 0, qmax)
    q = np.clip(np.rint(wg / safe[:, :, None]) + z[:, :, None], 0, qmax)
    # degenerate groups: constant c = min
    c = mn
    s_deg = np.where(c == 0.0, 1.0, np.abs(c))
    z_deg = np.where(c < 0.0, 1.0, 0.0)
    q_deg = np.where(c > 0.0, 1.0, 0.0)
    s_out = np.where(degenerate, s_deg, s64).astype(np.float16)
    z_out = np.where(degenerate, z_deg, z).astype(np.float16)
    q_out = np.where(degenerate[:, :, None], q_deg[:, :, None], q)
    return q_out.reshape(oc, ic).astype(np.uint8), s_out, z_out


def sq_decode(q: np.ndarray, s: np.ndarray, z: np.ndarray, group: int = 128) -> np.ndarray:
    """Exact decode w_hat = s * (q - z) in float64 (inverse of Eq. 2)."""
    oc, ic = q.shape
    qg = q.astype(np.float64).reshape(oc, ic // group, group)
    out = s.astype(np.float64)[:, :, None] * (qg - z.astype(np.float64)[:, :, None])
    return out.reshape(oc, ic)


# --------------------------------------------------------------------------
# Vector quantization, Section 3.2 Eq. 3
# --------------------------------------------------------------------------


def _nearest(vecs: np.ndarray, centres: np.ndarray, weights: np.ndarray | None = None) -> np.ndarray:
    """argmin_j ||v_i - C_j||^2 (Eq. 3); ties resolve to the lowest index.  With
    per-element weights X_ij^2 the distance is the term of Eq. 19 that vector i
    contributes, sum_d X_id^2 (v_id - C_jd)^2."""
    sq = (vecs[:, None, :] - centres[None, :, :]) ** 2
    if weights is not None:
        sq = weights[:, None, :] * sq
    return np.argmin(sq.sum(axis=2), axis=1)


def kmeans_tile(vecs: np.ndarray, entries: int, iters: int, rng: np.random.Generator,
                weights: np.ndarray | None = None, return_losses: bool = False):
    """k-means++ seeding followed by `iters` Lloyd iterations on one set of
    d-dimensional source vectors; returns (fp16 codebook [entries, d], idx).

    Seeding: first centre uniform over the vectors; each next centre drawn with
    probability proportional to the squared distance to the nearest centre so
    far (uniform when all distances are zero).  Lloyd: assign to nearest centre,
    move each centre to the (optionally weighted) mean of its members; an empty
    cluster keeps its previous centre.  Centres are then rounded to fp16 and the
    final assignment is taken against the rounded centres.

    With `weights` (X^2 of Section 4.2, one per vector or one per element) both
    Lloyd half-steps minimise the loss of Eq. 19: vectors go to the centre with
    the smallest weighted distance and a centre moves, per dimension, to the
    weighted mean of its members (a dimension whose member weights sum to zero
    keeps its value).  Seeding ignores the weights.
    """
    v = np.asarray(vecs, dtype=np.float64)
    n, d = v.shape
    wt = np.ones((n, 1)) if weights is None else np.asarray(weights, dtype=np.float64).reshape(n, -1)
    wa = None if weights is None else np.broadcast_to(wt, (n, d))
    centres = np.empty((entries, d))
    centres[0] = v[rng.integers(n)]
    dist = ((v - centres[0]) ** 2).sum(axis=1)
    for e in range(1, entries):
        tot = dist.sum()
        if tot > 0.0:
            pick = int(np.searchsorted(np.cumsum(dist), rng.random() * tot, side="right"))
            pick = min(pick, n - 1)
        else:
            pick = int(rng.integers(n))
        centres[e] = v[pick]
        dist = np.minimum(dist, ((v - centres[e]) ** 2).sum(axis=1))
    losses = []
    for _ in range(iters):
        idx = _nearest(v, centres, wa)
        if return_losses:
            losses.append(float((wt * (v - centres[idx]) ** 2).sum()))
        for dd in range(d):
            wcol = wt[:, dd] if wt.shape[1] == d else wt[:, 0]
            num = np.bincount(idx, weights=wcol * v[:, dd], minlength=entries)
            den = np.bincount(idx, weights=wcol, minlength=entries)
            upd = den > 0
            centres[upd, dd] = num[upd] / den[upd]
    cb16 = centres.astype(np.float16)
    idx = _nearest(v, cb16.astype(np.float64), wa)
    if return_losses:
        losses.append(float((wt * (v - cb16.astype(np.float64)[idx]) ** 2).sum()))
        return cb16, idx, losses
    return cb16, idx


def vq_encode(w16: np.ndarray, entries: int = 64, tile: int = 256, iters: int = 10, seed: int = 0):
    """VQ with 2-D vectors (two consecutive input-dim weights of one row, i.e. the
    row-major (m*n//d, d) reshape of Section 3.2) and one codebook per
    tile x tile block.  Returns codebooks float16 [oc/tile, ic/tile, entries, 2]
    and idx [oc, ic/2] (uint8 for <=256 entries)."""
    w = np.asarray(w16, dtype=np.float16)
    oc, ic = w.shape
    assert oc % tile == 0 and ic % tile == 0
    tr, tc = oc // tile, ic // tile
    cbs = np.zeros((tr, tc, entries, 2), dtype=np.float16)
    idx = np.zeros((oc, ic // 2), dtype=np.uint8 if entries <= 256 else np.uint16)
    rng = np.random.default_rng(seed)
    for i in range(tr):
        for j in range(tc):
            blk = w[i * tile:(i + 1) * tile, j * tile:(j + 1) * tile].astype(np.float64)
            cb, ix = kmeans_tile(blk.reshape(-1, 2), entries, iters, rng)
            cbs[i, j] = cb
            idx[i * tile:(i + 1) * tile, j * (tile // 2):(j + 1) * (tile // 2)] = ix.reshape(tile, tile // 2)
    return cbs, idx


def vq_decode(cbs: np.ndarray, idx: np.ndarray, tile: int = 256) -> np.ndarray:
    """Exact decode by table lookup: w_hat[i, 2p+e] = C_tile(i,p)[idx[i,p]][e]."""
    oc, half = idx.shape
    ic = half * 2
    out = np.empty((oc, ic), dtype=np.float64)
    tr, tc = cbs.shape[0], cbs.shape[1]
    th = tile // 2
    for i in range(tr):
        for j in range(tc):
            ix = idx[i * tile:(i + 1) * tile, j * th:(j + 1) * th].astype(np.int64)
            out[i * tile:(i + 1) * tile, j * tile:(j + 1) * tile] = (
                cbs[i, j].astype(np.float64)[ix].reshape(ix.shape[0], -1))
    return out


def mu_encode(mu16: np.ndarray, entries: int = 64, iters: int = 10, seed: int = 0,
              act_sq: np.ndarray | None = None):
    """VQ of one token-shift vector mu (a 1 x ic "matrix", Section 4.2): 2-D
    vectors, a single codebook.  With `act_sq` (X^2 of Eq. 19, same length as
    mu) the Lloyd means are weighted by it (the weighted k-means of Section 4.2).
    Returns codebook float16 [entries, 2], idx [ic/2]."""
    mu = np.asarray(mu16, dtype=np.float16).astype(np.float64).reshape(-1, 2)
    rng = np.random.default_rng(seed)
    wts = None if act_sq is None else np.asarray(act_sq, dtype=np.float64).reshape(-1, 2)
    cb, ix = kmeans_tile(mu, entries, iters, rng, weights=wts)
    return cb, ix.astype(np.uint8 if entries <= 256 else np.uint16)


def representative_activation(samples: np.ndarray, pct: float) -> np.ndarray:
    """Representative X of a batch of calibration activations (Section 4.2):
    every position's samples are first limited to the range between their
    pct-th and (100 - pct)-th percentiles (percentiles by linear interpolation
    between order statistics), then averaged.  samples: [S, n]; returns [n]
    float64.  pct = 0 is the plain mean the paper calls outlier-prone."""
    x = np.asarray(samples, dtype=np.float64)
    assert x.ndim == 2 and 0.0 <= pct < 50.0
    lo = np.percentile(x, pct, axis=0)
    hi = np.percentile(x, 100.0 - pct, axis=0)
    return np.clip(x, lo[None, :], hi[None, :]).mean(axis=0)


def mu_decode(cb: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """mu_hat[2p+e] = C[idx[p]][e], float64."""
    return cb.astype(np.float64)[idx.astype(np.int64)].reshape(-1)


# --------------------------------------------------------------------------
# Coarse-to-fine proxy, Section 4.1
# --------------------------------------------------------------------------


def proxy(w: np.ndarray, K: int = 4):
    """Coarse proxy P_c (Eqs. 5-9) and fine proxy P_f (Eqs. 10-17), literally:

        W' = sort(flatten(W));  G = W'[1:] - W'[:-1];  n = oc*ic - 1
        G' = G / sum(G);        H = -sum G' ln G'   (0 ln 0 := 0)
        P_c = ln n - H
        delta = G' - 1/n;       M_k = sum(delta^k)/n;  v_k = n^k / (k (k-1))
        P_f = sum_{k=2..K} v_k |M_k|

    A constant matrix (sum(G) == 0) has no defined G'; it returns (inf, inf).
    Returns (P_c, P_f) as Python floats.
    """
    flat = np.sort(np.asarray(w, dtype=np.float64).reshape(-1))
    g = flat[1:] - flat[:-1]
    n = g.size
    tot = g.sum()
    if not tot > 0.0:
        return math.inf, math.inf
    gp = g / tot
    nz = gp[gp > 0.0]
    h = -float((nz * np.log(nz)).sum())
    pc = math.log(n) - h
    delta = gp - 1.0 / n
    pf = 0.0
    for k in range(2, K + 1):
        mk = float((delta ** k).sum()) / n
        vk = float(n) ** k / (k * (k - 1))
        pf += vk * abs(mk)
    return pc, pf


def proxy_segments(w: np.ndarray, seg_rows: int, seg_cols: int, K: int = 4):
    """The proxy of Section 4.1 applied to every seg_rows x seg_cols tile of a matrix instead of
    the whole matrix (the paper's limitations paragraph: finer granularity than one decision per
    matrix): tile (i, j) covers rows i*seg_rows.. and columns j*seg_cols.., smaller at the right
    and bottom edges; a tile with fewer than two elements has no gaps and returns (inf, inf).
    Returns (P_c, P_f) arrays of shape [ceil(oc / seg_rows), ceil(ic / seg_cols)]."""
    w = np.asarray(w, dtype=np.float64)
    oc, ic = w.shape
    gy, gx = -(-oc // seg_rows), -(-ic // seg_cols)
    pc = np.full((gy, gx), math.inf)
    pf = np.full((gy, gx), math.inf)
    for i in range(gy):
        for j in range(gx):
            t = w[i * seg_rows:(i + 1) * seg_rows, j * seg_cols:(j + 1) * seg_cols]
            if t.size >= 2:
                pc[i, j], pf[i, j] = proxy(t, K)
    return pc, pf


def proxy_taylor_signed(w: np.ndarray, K: int) -> float:
    """Signed Taylor sum of Eq. 14/15: sum_k (-1)^k v_k M_k (approximates P_c near uniform)."""
    flat = np.sort(np.asarray(w, dtype=np.float64).reshape(-1))
    g = flat[1:] - flat[:-1]
    n = g.size
    gp = g / g.sum()
    delta = gp - 1.0 / n
    tot = 0.0
    for k in range(2, K + 1):
        mk = float((delta ** k).sum()) / n
        tot += (-1.0) ** k * float(n) ** k / (k * (k - 1)) * mk
    return tot


def proxy_family(w: np.ndarray) -> dict:
    """The simpler statistics of the normalised gaps G' that the ablation of Section 5.3 puts in
    the proxy's place (Variance, Coefficient of Variation, Range, Mean Absolute Deviation, and the
    information entropy alone), each in its textbook form on the n values G'_i (mean 1/n):

        variance = sum (G' - 1/n)^2 / n        cv = sqrt(variance) / (1/n)
        range    = max G' - min G'             mad = sum |G' - 1/n| / n
        ie       = -sum G' ln G'   (0 ln 0 := 0; P_c = ln n - ie)

    A constant matrix returns inf for all five."""
    flat = np.sort(np.asarray(w, dtype=np.float64).reshape(-1))
    g = flat[1:] - flat[:-1]
    n = g.size
    tot = g.sum()
    if not tot > 0.0:
        return {k: math.inf for k in ("variance", "cv", "range", "mad", "ie")}
    gp = g / tot
    mean = 1.0 / n
    var = float(((gp - mean) ** 2).sum()) / n
    nz = gp[gp > 0.0]
    return {"variance": var, "cv": math.sqrt(var) / mean, "range": float(gp.max() - gp.min()),
            "mad": float(np.abs(gp - mean).sum()) / n, "ie": -float((nz * np.log(nz)).sum())}


def quant_sse(w: np.ndarray, w_hat: np.ndarray) -> float:
    """Sum of squared quantization errors sum (w - w_hat)^2 in float64: the quantity the "MSE"
    selector of Section 5.3 compares between the SQ and the VQ coding of a matrix."""
    d = np.asarray(w, dtype=np.float64) - np.asarray(w_hat, dtype=np.float64)
    return float((d * d).sum())


def tau_for_fraction(values, sq_fraction: float) -> float:
    """Threshold that sends the given fraction of the matrices to scalar quantization under
    "SQ iff value < tau" (Section 5.1 sets the thresholds so that nine tenths of the layers use SQ):
    with the M values sorted and k = round(sq_fraction * M), tau lies halfway between the k-th and
    the (k+1)-th smallest; k = 0 gives -inf and k = M gives +inf."""
    v = np.sort(np.asarray(values, dtype=np.float64))
    m = v.size
    k = int(np.rint(sq_fraction * m))
    if k <= 0:
        return -math.inf
    if k >= m:
        return math.inf
    return 0.5 * (float(v[k - 1]) + float(v[k]))


def select(pc: float, pf: float, tau_c: float, tau_f: float) -> int:
    """phi of Eq. 18: 1 (scalar quantization) iff P_c < tau_c and P_f < tau_f, else 0 (VQ)."""
    return 1 if (pc < tau_c and pf < tau_f) else 0


# --------------------------------------------------------------------------
# Runtime math, Appendix A.1
# --------------------------------------------------------------------------


def token_shift(x: np.ndarray, x_prev: np.ndarray, mu_hat: np.ndarray) -> np.ndarray:
    """x_mix = x + (x_prev - x) * mu_hat, float64.  This is Eq. 20's
    mu_p*x_t + (1-mu_p)*x_{t-1} with mu_p = 1 - mu_hat (the RWKV-6 way of
    writing the same interpolation)."""
    x = np.asarray(x, dtype=np.float64)
    xp = np.asarray(x_prev, dtype=np.float64)
    return x + (xp - x) * np.asarray(mu_hat, dtype=np.float64)[None, :]


def prefill_prev(X: np.ndarray, x_prev0: np.ndarray | None) -> np.ndarray:
    """Previous-token matrix for a sequence: row t is X[t-1]; row 0 is x_prev0 (zeros if None)."""
    X = np.asarray(X, dtype=np.float64)
    P = np.empty_like(X)
    P[1:] = X[:-1]
    P[0] = 0.0 if x_prev0 is None else np.asarray(x_prev0, dtype=np.float64)
    return P


def gemv(w_hat: np.ndarray, x_mix: np.ndarray) -> np.ndarray:
    """y[b, i] = sum_j w_hat[i, j] * x_mix[b, j] in float64 (the W.(...) products of Eqs. 20-22 and 24-27)."""
    return np.asarray(x_mix, dtype=np.float64) @ np.asarray(w_hat, dtype=np.float64).T


def tolerance(w_hat: np.ndarray, x_mix: np.ndarray, rel: float = 2e-3) -> np.ndarray:
    """Per-element bound rel * ||w_hat_row||_2 * ||x_mix[b]||_2, shape [B, oc]."""
    wn = np.sqrt((np.asarray(w_hat, dtype=np.float64) ** 2).sum(axis=1))
    xn = np.sqrt((np.asarray(x_mix, dtype=np.float64) ** 2).sum(axis=1))
    return rel * xn[:, None] * wn[None, :]


def sigmoid(x: np.ndarray) -> np.ndarray:
    """sigma(x) = 1 / (1 + exp(-x)), float64."""
    return 1.0 / (1.0 + np.exp(-np.asarray(x, dtype=np.float64)))


def wkv_literal(ks: np.ndarray, vs: np.ndarray, u: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Eq. 23 written out for the LAST token of a history: ks, vs are [T, d] (tokens 1..T = t),

        wkv_t = ( sum_{i<t} f(i) * v_i + exp(u + k_t) * v_t ) / ( sum_{i<t} f(i) + exp(u + k_t) ),
        f(i)  = exp( -(t - 1 - i) * w + k_i ),

    element-wise over the d channels, float64.  Returns [d]."""
    ks, vs = np.asarray(ks, dtype=np.float64), np.asarray(vs, dtype=np.float64)
    u, w = np.asarray(u, dtype=np.float64), np.asarray(w, dtype=np.float64)
    t = ks.shape[0]
    num = np.exp(u + ks[t - 1]) * vs[t - 1]
    den = np.exp(u + ks[t - 1])
    for i in range(1, t):                       # token numbers 1 .. t-1
        f = np.exp(-(t - 1 - i) * w + ks[i - 1])
        num = num + f * vs[i - 1]
        den = den + f
    return num / den


def wkv_step(a: np.ndarray, b: np.ndarray, k: np.ndarray, v: np.ndarray, u: np.ndarray, w: np.ndarray):
    """One token of Eq. 23 as a recurrence over the two history sums a_{t-1} = sum_{i<t} f(i) v_i and
    b_{t-1} = sum_{i<t} f(i):  wkv_t = (a + e^{u+k} v) / (b + e^{u+k});  the sums for the next token are
    a' = e^{-w} a + e^{k} v,  b' = e^{-w} b + e^{k}  (every f(i) gains the factor e^{-w}, token t joins
    with f = e^{k_t}).  All arrays [B, d] or [d], float64.  Returns (wkv, a', b')."""
    a, b, k, v = (np.asarray(z, dtype=np.float64) for z in (a, b, k, v))
    u, w = np.asarray(u, dtype=np.float64), np.asarray(w, dtype=np.float64)
    e = np.exp(u + k)
    wkv = (a + e * v) / (b + e)
    return wkv, np.exp(-w) * a + np.exp(k) * v, np.exp(-w) * b + np.exp(k)


def time_mix_gate(r: np.ndarray, wkv: np.ndarray) -> np.ndarray:
    """Input of the output projection, Eq. 24: sigma(r) * wkv."""
    return sigmoid(r) * np.asarray(wkv, dtype=np.float64)


def relu_squared(k: np.ndarray) -> np.ndarray:
    """Input of the channel-mix value projection, Eq. 27: max(k', 0)^2."""
    return np.maximum(np.asarray(k, dtype=np.float64), 0.0) ** 2


def channel_mix_gate(r: np.ndarray, y: np.ndarray) -> np.ndarray:
    """Output of channel mixing, Eq. 27: sigma(r') * y with y = W'_v . max(k', 0)^2."""
    return sigmoid(r) * np.asarray(y, dtype=np.float64)


def rms_normalize(x: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """Row-wise x / sqrt(mean(x^2) + eps), float64.  Not printed in the paper's appendix: the chained-block
    workload normalises the inputs of time mixing and of channel mixing this way (the places where the
    models the paper quantizes normalise), because a chain of the printed blocks alone does not keep its
    activations in range."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)

