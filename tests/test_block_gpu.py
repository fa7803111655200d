"""GPU parity of the element-wise operators between the projections of an RWKV block (Appendix A.1 Eq. 23 WKV,
Eq. 24 sigmoid gate, Eq. 27 squared ReLU and output gate), fused into the input stage of the persistent decode
step: a two-layer block chain is run for several tokens and every product, every recurrence state and every
previous-token state is checked against the oracle, each from the GPU's own upstream values (so an error
cannot hide behind the one before it)."""
import numpy as np
import pytest
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs

pytestmark = pytest.mark.gpu


class _Mat:
    def __init__(self, seed, oc, ic, method, std):
        w = (np.random.default_rng(seed).standard_normal((oc, ic)) * std).astype(np.float16)
        bits = 3 if method == B.RWKVQ_SQ else 6
        blob = B.rwkvq_pack(w, oc, ic, method, bits, kmeans_iters=2, seed=seed)
        c = blob.export_codes()
        self.w_hat = orc.sq_decode(c["q"], c["scale"], c["zero"]) if method == B.RWKVQ_SQ else orc.vq_decode(c["codebook"], c["q"])
        self.desc, self.dev, self.oc, self.ic = blob.desc, blob.to_device(), oc, ic


class _Mu:
    def __init__(self, seed, ic):
        blob = B.rwkvq_pack(inputs.gen_mu(seed, ic).reshape(1, -1), 1, ic, B.RWKVQ_VQ, 6, seed=seed)
        c = blob.export_codes()
        self.mu_hat = orc.mu_decode(c["codebook"], c["q"])
        self.desc, self.dev = blob.desc, blob.to_device()


def _f16(a):
    return np.asarray(a, dtype=np.float64).astype(np.float16).astype(np.float64)


def _build(d, h, layers, Bn, seed):
    """Ops of `layers` blocks: per block R, K, V (stage 0), O (1), cm_k and cm_r (2), cm_v (3)."""
    dev = "cuda"
    z32 = lambda *s: torch.zeros(s, dtype=torch.float32, device=dev)
    z16 = lambda *s: torch.zeros(s, dtype=torch.float16, device=dev)
    rng = np.random.default_rng(seed)
    x0 = z16(Bn, d)
    ops, entries = [], []
    prev = None           # (y_cm_r, y_cm_v) of the block before
    for l in range(layers):
        s0 = seed * 100 + l * 10
        m = {"R": _Mat(s0 + 1, d, d, B.RWKVQ_SQ, 0.08), "K": _Mat(s0 + 2, d, d, B.RWKVQ_VQ, 0.08),
             "V": _Mat(s0 + 3, d, d, B.RWKVQ_SQ, 0.08), "O": _Mat(s0 + 4, d, d, B.RWKVQ_SQ, 0.08),
             "cK": _Mat(s0 + 5, h, d, B.RWKVQ_SQ, 0.08), "cR": _Mat(s0 + 6, d, d, B.RWKVQ_SQ, 0.08),
             "cV": _Mat(s0 + 7, d, h, B.RWKVQ_VQ if l == 0 else B.RWKVQ_SQ, 0.08)}
        mu = {n: _Mu(s0 + 20 + i, d) for i, n in enumerate(("R", "K", "V", "cK", "cR"))}
        y = {n: z32(Bn, m[n].oc) for n in m}
        xs = {n: z16(Bn, d) for n in mu}                      # previous-token input, one per product
        st = {"a": z32(Bn, d), "b": z32(Bn, d), "p": torch.full((Bn, d), -1e30, dtype=torch.float32, device=dev),
              "u": torch.from_numpy((rng.standard_normal(d) * 0.3).astype(np.float32)).to(dev),
              "w": torch.from_numpy(rng.uniform(0.05, 1.0, d).astype(np.float32)).to(dev),
              "gain": torch.full((1,), 0.5 + 0.25 * l, dtype=torch.float32, device=dev)}
        blk = dict(m=m, mu=mu, y=y, xs=xs, st=st, prev=prev)
        for n in ("R", "K", "V"):
            if prev is None:
                xin = dict(kind=B.RWKVQ_IN_BUFFER, xprev_out=xs[n])
                e = dict(x=x0)
            else:
                xin = dict(kind=B.RWKVQ_IN_F32, src=prev[1], gate=prev[0], xprev_out=xs[n], rmsnorm=True)
                e = dict(x=None)
            e.update(desc=m[n].desc, W=m[n].dev, mu_desc=mu[n].desc, mu=mu[n].dev, xprev=xs[n], y=y[n], stage=4 * l, **{"in": xin})
            entries.append(e)
        entries.append(dict(desc=m["O"].desc, W=m["O"].dev, x=None, y=y["O"], stage=4 * l + 1,
                            **{"in": dict(kind=B.RWKVQ_IN_WKV, src=y["R"], k=y["K"], v=y["V"], state_a=st["a"], state_b=st["b"],
                                          state_p=st["p"], u=st["u"], w=st["w"], scale=st["gain"])}))
        for n in ("cK", "cR"):
            entries.append(dict(desc=m[n].desc, W=m[n].dev, mu_desc=mu[n].desc, mu=mu[n].dev, x=None, xprev=xs[n], y=y[n],
                                stage=4 * l + 2, **{"in": dict(kind=B.RWKVQ_IN_F32, src=y["O"], xprev_out=xs[n], rmsnorm=(n == "cK"))}))
        entries.append(dict(desc=m["cV"].desc, W=m["cV"].dev, x=None, y=y["cV"], stage=4 * l + 3,
                            **{"in": dict(kind=B.RWKVQ_IN_RELU2, src=y["cK"])}))
        prev = (y["cR"], y["cV"])
        ops.append(blk)
    return x0, ops, entries


def _np(t):
    return t.detach().double().cpu().numpy()


def _check_product(name, mat, x_ref, y_dev):
    ref, tol = orc.gemv(mat.w_hat, x_ref), orc.tolerance(mat.w_hat, x_ref)
    got = _np(y_dev)
    assert np.isfinite(got).all(), name
    err = np.abs(got - ref)
    assert (err <= tol + 1e-30).all(), f"{name}: max err/tol {float((err / np.maximum(tol, 1e-300)).max())}"


@pytest.mark.parametrize("Bn", [1, 3, 8, 16])
def test_block_chain_matches_oracle_token_by_token(Bn):
    d, h, layers = 256, 512, 2
    x0, blocks, entries = _build(d, h, layers, Bn, seed=Bn)
    ops = B.make_ops(entries)
    plan = torch.zeros(B.rwkvq_step_plan_bytes(ops, Bn), dtype=torch.uint8, device="cuda")
    B.rwkvq_step_plan(ops, Bn, plan)
    for token in range(4):
        x_host = inputs.gen_activation(1000 + 17 * Bn + token, Bn, d, 4).astype(np.float16)
        x0.copy_(torch.from_numpy(x_host).cuda())
        # states before the step
        before = [dict(xs={n: _np(t) for n, t in blk["xs"].items()},
                       a=_np(blk["st"]["a"]), b=_np(blk["st"]["b"]), p=_np(blk["st"]["p"])) for blk in blocks]
        B.rwkvq_step_run(plan)
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        for l, blk in enumerate(blocks):
            m, mu, y, st, bf = blk["m"], blk["mu"], blk["y"], blk["st"], before[l]
            # input of the time-mix projections: the token itself, or the gated output of the block before (Eq. 27)
            if blk["prev"] is None:
                x_t = x_host.astype(np.float64)
            else:
                x_t = _f16(orc.rms_normalize(orc.channel_mix_gate(_np(blk["prev"][0]), _np(blk["prev"][1]))))
            for n in ("R", "K", "V"):
                _check_product(f"token {token} layer {l} {n}", m[n], orc.token_shift(x_t, bf["xs"][n], mu[n].mu_hat), y[n])
                got_state = _np(blk["xs"][n])
                assert (np.abs(got_state - x_t) <= 2.0 ** -10 * np.abs(x_t) + 1e-7).all()    # within one fp16 step of x_t
            # Eq. 23 from the history sums before the step (stored scaled by e^{-p}), Eq. 24 gate
            a_true, b_true = bf["a"] * np.exp(bf["p"]), bf["b"] * np.exp(bf["p"])
            u, w = _np(st["u"]), _np(st["w"])
            wkv, a_new, b_new = orc.wkv_step(a_true, b_true, _np(y["K"]), _np(y["V"]), u, w)
            gain = float(st["gain"][0])
            _check_product(f"token {token} layer {l} O", m["O"], _f16(gain * orc.time_mix_gate(_np(y["R"]), wkv)), y["O"])
            ga, gb = _np(st["a"]) * np.exp(_np(st["p"])), _np(st["b"]) * np.exp(_np(st["p"]))
            # fp32 recurrence: relative to the magnitudes that are added (the numerator sum can cancel)
            a_scale = np.exp(-w) * np.abs(a_true) + np.exp(_np(y["K"])) * np.abs(_np(y["V"]))
            assert (np.abs(ga - a_new) <= 2e-5 * a_scale + 1e-30).all() and np.allclose(gb, b_new, rtol=2e-5, atol=1e-30)
            for n in ("cK", "cR"):       # cm_k reads the normalised output of time mixing, cm_r the plain one
                x_c = _f16(orc.rms_normalize(_np(y["O"]))) if n == "cK" else _f16(_np(y["O"]))
                _check_product(f"token {token} layer {l} {n}", m[n], orc.token_shift(x_c, bf["xs"][n], mu[n].mu_hat), y[n])
                assert (np.abs(_np(blk["xs"][n]) - x_c) <= 2.0 ** -10 * np.abs(x_c) + 1e-7).all()
            _check_product(f"token {token} layer {l} cV", m["cV"], _f16(orc.relu_squared(_np(y["cK"]))), y["cV"])
    B.rwkvq_step_plan_release(plan)


def test_block_first_token_and_argument_checks():
    # first token of a sequence: the history is empty, so wkv = v and the output projection sees sigmoid(r) * v
    Bn, d, h = 2, 256, 512
    x0, blocks, entries = _build(d, h, 1, Bn, seed=77)
    ops = B.make_ops(entries)
    plan = torch.zeros(B.rwkvq_step_plan_bytes(ops, Bn), dtype=torch.uint8, device="cuda")
    B.rwkvq_step_plan(ops, Bn, plan)
    x0.copy_(torch.from_numpy(inputs.gen_activation(5, Bn, d, 4).astype(np.float16)).cuda())
    B.rwkvq_step_run(plan)
    torch.cuda.synchronize()
    blk = blocks[0]
    y = blk["y"]
    _check_product("first token O", blk["m"]["O"], _f16(0.5 * orc.sigmoid(_np(y["R"])) * _np(y["V"])), y["O"])
    B.rwkvq_step_plan_release(plan)
    # a WKV input without its state, and an unknown kind, are refused before anything is planned
    bad = [dict(e) for e in entries]
    bad[3] = dict(bad[3], **{"in": dict(kind=B.RWKVQ_IN_WKV, src=y["R"], k=y["K"], v=y["V"])})
    assert B.rwkvq_step_plan_bytes(B.make_ops(bad), Bn) == 0
    bad = [dict(e) for e in entries]
    bad[6] = dict(bad[6], **{"in": dict(kind=9, src=y["cK"])})
    assert B.rwkvq_step_plan_bytes(B.make_ops(bad), Bn) == 0


def _decode(st, op):
    codes, mu_codes = st.host_codes(op)
    w_hat = orc.sq_decode(codes["q"], codes["scale"], codes["zero"]) if op.method == B.RWKVQ_SQ else orc.vq_decode(codes["codebook"], codes["q"])
    mu_hat = orc.mu_decode(mu_codes["codebook"], mu_codes["q"]) if mu_codes is not None else None
    return w_hat, mu_hat


@pytest.mark.parametrize("batch", [1, 16])
def test_chained_blocks_at_7b_width_sampled(batch):
    """The chain bench.py times (BlockStack), two blocks of the 7B-class width: after two tokens, one product of
    every kind of input operator is recomputed by the oracle from the values the GPU holds upstream."""
    from paper_2505_03803_b200 import stack as stack_mod
    st = stack_mod.BlockStack(4096, 14336, 2, 64, batch, n_outliers=8, tag="c3_7b", kmeans_iters=2)
    by = {(o.layer, o.name): o for o in st.ops}
    for token in range(2):
        st.set_token(50 + token)
        prev_R1 = _np(by[(1, "R")].xprev)
        prev_ck0 = _np(by[(0, "cm_k")].xprev)
        a0, b0, p0 = (_np(st.states[0][k]) for k in ("a", "b", "p"))
        st.run_step_host()
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
    y = {k: _np(o.y) for k, o in by.items()}
    assert all(np.isfinite(v).all() for v in y.values())
    # block 1, R: gated and normalised output of block 0 (Eq. 27), token-shift mix with the token before
    w_hat, mu_hat = _decode(st, by[(1, "R")])
    x_t = _f16(orc.rms_normalize(orc.channel_mix_gate(y[(0, "cm_r")], y[(0, "cm_v")])))
    _check_product("block 1 R", type("M", (), {"w_hat": w_hat}), orc.token_shift(x_t, prev_R1, mu_hat), by[(1, "R")].y)
    # block 0, O: WKV (Eq. 23) from the history before the second token, sigmoid gate (Eq. 24)
    w_hat, _ = _decode(st, by[(0, "O")])
    wkv, _, _ = orc.wkv_step(a0 * np.exp(p0), b0 * np.exp(p0), y[(0, "K")], y[(0, "V")], _np(st.states[0]["u"]), _np(st.states[0]["w"]))
    _check_product("block 0 O", type("M", (), {"w_hat": w_hat}), _f16(orc.time_mix_gate(y[(0, "R")], wkv)), by[(0, "O")].y)
    # block 0, cm_k: normalised output of time mixing with its own token shift; cm_v: squared ReLU (Eq. 27)
    w_hat, mu_hat = _decode(st, by[(0, "cm_k")])
    x_c = _f16(orc.rms_normalize(y[(0, "O")]))
    _check_product("block 0 cm_k", type("M", (), {"w_hat": w_hat}), orc.token_shift(x_c, prev_ck0, mu_hat), by[(0, "cm_k")].y)
    w_hat, _ = _decode(st, by[(1, "cm_v")])
    _check_product("block 1 cm_v", type("M", (), {"w_hat": w_hat}), _f16(orc.relu_squared(y[(1, "cm_k")])), by[(1, "cm_v")].y)
