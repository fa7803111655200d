"""GPU parity of the whole-step persistent launch (rwkvq_step_plan / rwkvq_step_run) against the
oracle, product by product."""
import numpy as np
import pytest
import torch

from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _build_ops(d, h, layers, Bn, bits, seed, all_method=None):
    """Logical codes drawn at random (valid by construction), packed by the library."""
    ops = []
    k = 0
    for l in range(layers):
        for (name, oc, ic, has_mu, stage) in inputs.layer_shapes(d, h):
            k += 1
            use_sq = (k % 3 != 0) if all_method is None else (all_method == B.RWKVQ_SQ)
            W = H.pack_sq(H.random_sq_codes(seed + k, oc, ic)) if use_sq else H.pack_vq(H.random_vq_codes(seed + k, oc, ic, bits), bits)
            mu = H.pack_mu(H.random_mu_codes(seed + 100 + k, ic, bits), bits) if has_mu else None
            x, xp = inputs.gen_activation_pair(seed + 200 + k, Bn, ic, n_outliers=4)
            x16, xp16 = x.astype(np.float16), xp.astype(np.float16)
            e = dict(W=W, mu=mu, x16=x16, xp16=xp16, stage=4 * l + stage,
                     xd=torch.from_numpy(x16).cuda(), xpd=torch.from_numpy(xp16).cuda() if has_mu else None,
                     y=torch.full((Bn, oc), float("nan"), dtype=torch.float32, device="cuda"))
            ops.append(e)
    ops.sort(key=lambda e: e["stage"])
    return ops


def _plan(ops, Bn):
    arr = B.make_ops([dict(desc=e["W"].desc, W=e["W"].dev, mu_desc=None if e["mu"] is None else e["mu"].desc,
                           mu=None if e["mu"] is None else e["mu"].dev, x=e["xd"], xprev=e["xpd"], y=e["y"],
                           stage=e["stage"]) for e in ops])
    n = B.rwkvq_step_plan_bytes(arr, Bn)
    assert n > 0
    plan = torch.zeros(n, dtype=torch.uint8, device="cuda")
    B.rwkvq_step_plan(arr, Bn, plan)
    return plan


def _check(ops, Bn):
    worst = 0.0
    for e in ops:
        y = e["y"].double().cpu().numpy()
        ref, tol = H.reference(e["W"], e["mu"], e["x16"], e["xp16"])
        err = np.abs(y - ref)
        assert np.isfinite(y).all()
        ratio = float((err / tol).max())
        worst = max(worst, ratio)
        assert (err <= tol).all(), f"stage {e['stage']}: max err/tol = {ratio}"
    return worst


@pytest.mark.parametrize("Bn,bits", [(1, 6), (8, 6), (16, 8), (3, 8), (2, 6), (4, 6), (7, 8), (9, 6), (12, 8)])
def test_step_matches_oracle_small_stack(Bn, bits):
    ops = _build_ops(512, 1280, 2, Bn, bits, seed=10 * Bn + bits)   # h = 5 column tiles: odd tile count
    plan = _plan(ops, Bn)
    for rep in range(3):          # outputs are cleared and recomputed on every run
        B.rwkvq_step_run(plan)
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        _check(ops, Bn)


@pytest.mark.parametrize("method", [B.RWKVQ_SQ, B.RWKVQ_VQ])
def test_step_matches_oracle_1p6b_layer(method):
    ops = _build_ops(2048, 7168, 1, 1, 6, seed=77, all_method=method)
    plan = _plan(ops, 1)
    B.rwkvq_step_run(plan)
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 0
    _check(ops, 1)


@pytest.mark.parametrize("Bn", [1, 5, 16])
def test_step_ragged_sq_shapes(Bn):
    # d = 384, h = 896: row counts that end in a half unit (one 128-row chunk) and input lengths
    # whose last 256-column tile is half empty
    ops = _build_ops(384, 896, 2, Bn, 6, seed=300 + Bn, all_method=B.RWKVQ_SQ)
    plan = _plan(ops, Bn)
    for rep in range(2):
        B.rwkvq_step_run(plan)
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        _check(ops, Bn)


def test_step_agrees_with_single_product_calls():
    ops = _build_ops(512, 1280, 1, 8, 6, seed=5)
    plan = _plan(ops, 8)
    B.rwkvq_step_run(plan)
    torch.cuda.synchronize()
    for e in ops:
        y1 = H.run_gemv(e["W"], e["mu"], e["x16"], e["xp16"])
        _, tol = H.reference(e["W"], e["mu"], e["x16"], e["xp16"])
        assert (np.abs(e["y"].double().cpu().numpy() - y1) <= tol).all()


def test_step_rejects_bad_plans():
    ops = _build_ops(512, 1280, 1, 1, 6, seed=6)
    plan = _plan(ops, 1)
    with pytest.raises(B.RwkvqError):
        B.rwkvq_step_run(plan[256:])         # not the buffer a plan was written to
    arr = B.make_ops([dict(desc=e["W"].desc, W=e["W"].dev, mu_desc=None, mu=None, x=e["xd"], xprev=None,
                           y=e["y"].half(), stage=e["stage"]) for e in ops[:1]])
    assert B.rwkvq_step_plan_bytes(arr, 1) == 0   # fp16 outputs are not supported by the step launch


@pytest.mark.parametrize("Bn,layout", [(4, "packed"), (4, "spread"), (16, "spread"), (1, "spread"), (8, "reversed")])
def test_step_run_host_matches_oracle(Bn, layout):
    """rwkvq_step_run_host (the call behind the benchmark's end-to-end figure): activations come from
    pinned host memory, results go back to pinned host memory, compared with the oracle there.
    "packed": small arenas, the copies run before and after the step.  "spread": the same products
    3 MB apart in arenas of tens of MB, so that the activations arrive in several chunks while the step
    runs and the outputs leave in several groups behind their stage barriers.  "reversed": outputs laid
    out against the order of the stages, which the call must answer with one copy at the end."""
    ops = _build_ops(512, 1280, 2, Bn, 6, seed=91 + Bn)
    # one arena for the activations and one for the outputs, as the stack runner lays them out
    gap = 0 if layout == "packed" else 3 << 20
    def al(n):
        return (n + 255) // 256 * 256 + gap
    act_off, y_off, slots = 0, 0, []
    for e in ops:
        xo = act_off; act_off += al(e["x16"].nbytes)
        po = None
        if e["mu"] is not None:
            po = act_off; act_off += al(e["xp16"].nbytes)
        slots.append([xo, po, y_off]); y_off += al(Bn * e["W"].oc * 4)
    if layout == "reversed":
        for sl, e in zip(slots, ops):
            sl[2] = y_off - sl[2] - al(Bn * e["W"].oc * 4)
    act_host = torch.zeros(act_off, dtype=torch.uint8).pin_memory()
    y_host = torch.zeros(y_off, dtype=torch.uint8).pin_memory()
    act_dev = torch.zeros(act_off, dtype=torch.uint8, device="cuda")
    y_dev = torch.full((y_off // 4,), float("nan"), dtype=torch.float32, device="cuda").view(torch.uint8)
    an = act_host.numpy()
    for e, (xo, po, yo) in zip(ops, slots):
        an[xo:xo + e["x16"].nbytes] = e["x16"].reshape(-1).view(np.uint8)
        e["xd"] = act_dev[xo:xo + e["x16"].nbytes].view(torch.float16).view(Bn, -1)
        if po is not None:
            an[po:po + e["xp16"].nbytes] = e["xp16"].reshape(-1).view(np.uint8)
            e["xpd"] = act_dev[po:po + e["xp16"].nbytes].view(torch.float16).view(Bn, -1)
        e["y"] = y_dev[yo:yo + Bn * e["W"].oc * 4].view(torch.float32).view(Bn, e["W"].oc)
    plan = _plan(ops, Bn)
    for rep in range(2):
        y_host.zero_()
        B.rwkvq_step_run_host(plan, act_host, act_dev, y_dev, y_host)
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        assert torch.equal(act_dev.cpu(), act_host)                      # the inputs went through the call
        yn = y_host.numpy()
        for e, (xo, po, yo) in zip(ops, slots):
            y = yn[yo:yo + Bn * e["W"].oc * 4].view(np.float32).reshape(Bn, -1).astype(np.float64)
            ref, tol = H.reference(e["W"], e["mu"], e["x16"], e["xp16"])
            assert np.isfinite(y).all() and (np.abs(y - ref) <= tol).all()
    B.rwkvq_step_plan_release(plan)
    with pytest.raises(B.RwkvqError):
        B.rwkvq_step_run(plan)                                           # the record of the plan is gone


def test_bounded_waits_run_out_and_the_plan_recovers():
    """No wait inside the step kernel is unbounded.  With a barrier target that can never be met
    (wait_skew) and a small poll limit every CTA gives up at its first stage barrier, the kernel
    returns, the status word says ETIMEOUT; after the status has been read the next run clears the
    barrier counters and matches the oracle again.  Nothing traps, faults or hangs."""
    for Bn in (1, 8):
        ops = _build_ops(512, 1280, 2, Bn, 6, seed=40 + Bn)
        plan = _plan(ops, Bn)
        B.rwkvq_step_run(plan)
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        _check(ops, Bn)
        B.rwkvq_step_set_wait(plan, poll_limit=2000, wait_skew=1)
        B.rwkvq_step_run(plan)
        torch.cuda.synchronize()                                         # the kernel returns by itself
        assert B.rwkvq_device_status() == 8                              # RWKVQ_ETIMEOUT, and the word is cleared
        assert B.rwkvq_device_status() == 0
        B.rwkvq_step_set_wait(plan, poll_limit=0, wait_skew=0)           # defaults again
        for rep in range(2):
            for e in ops:
                e["y"].fill_(float("nan"))
            B.rwkvq_step_run(plan)
            torch.cuda.synchronize()
            assert B.rwkvq_device_status() == 0
            _check(ops, Bn)


@pytest.mark.parametrize("Bn", [1, 8, 16])
def test_step_output_rows_end_inside_a_unit(Bn):
    """Row counts that end inside a 256-row unit (272 = one unit and one record) and inside a 128-row chunk
    (144): the 16-byte reductions of the flush stop at the last row; nothing beyond the outputs is written.
    An output that does not start on a 16-byte boundary is refused by the plan."""
    ops = []
    for k, (oc, ic) in enumerate([(272, 384), (144, 640), (256, 512), (272, 384)]):
        W = H.pack_sq(H.random_sq_codes(900 + 10 * Bn + k, oc, ic)) if k != 2 else H.pack_vq(H.random_vq_codes(900 + 10 * Bn + k, oc, ic, 6), 6)
        mu = H.pack_mu(H.random_mu_codes(950 + 10 * Bn + k, ic, 6), 6) if k % 2 == 0 else None
        x, xp = inputs.gen_activation_pair(990 + 10 * Bn + k, Bn, ic, n_outliers=4)
        x16, xp16 = x.astype(np.float16), xp.astype(np.float16)
        buf = torch.full((Bn * oc + 8,), float("nan"), dtype=torch.float32, device="cuda")
        y = buf[4:4 + Bn * oc].view(Bn, oc)
        ops.append(dict(W=W, mu=mu, x16=x16, xp16=xp16, stage=k // 2, xd=torch.from_numpy(x16).cuda(),
                        xpd=torch.from_numpy(xp16).cuda() if mu is not None else None, y=y, buf=buf))
    plan = _plan(ops, Bn)
    for _ in range(2):
        B.rwkvq_step_run(plan)
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        _check(ops, Bn)
    for e in ops:      # nothing outside the outputs was touched
        assert torch.isnan(e["buf"][:4]).all() and torch.isnan(e["buf"][4 + e["y"].numel():]).all()
    e = ops[0]
    bad = e["buf"][1:1 + Bn * e["W"].oc].view(Bn, e["W"].oc)
    arr = B.make_ops([dict(desc=e["W"].desc, W=e["W"].dev, mu_desc=e["mu"].desc, mu=e["mu"].dev, x=e["xd"], xprev=e["xpd"],
                           y=bad, stage=0)])
    assert B.rwkvq_step_plan_bytes(arr, Bn) == 0
