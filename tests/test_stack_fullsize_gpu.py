"""Parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times
(one rwkvq_step_run over the whole stack): sampled products are compared with the fp64 oracle
computed from the logical codes the packer exported."""
import numpy as np
import pytest
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import stack as stack_mod

pytestmark = pytest.mark.gpu


def _oracle_product(st, op):
    codes, mu_codes = st.host_codes(op)
    if op.method == B.RWKVQ_SQ:
        w_hat = orc.sq_decode(codes["q"], codes["scale"], codes["zero"])
    else:
        w_hat = orc.vq_decode(codes["codebook"], codes["q"])
    x = op.x.cpu().numpy().astype(np.float64)
    if op.has_mu:
        mu_hat = orc.mu_decode(mu_codes["codebook"], mu_codes["q"])
        x = orc.token_shift(x, op.xprev.cpu().numpy().astype(np.float64), mu_hat)
    return orc.gemv(w_hat, x), orc.tolerance(w_hat, x)


@pytest.mark.parametrize("name,batch,quantizer,weights", [
    ("c2_1p6b", 1, "host", "host"), ("c3_7b", 8, "host", "host"), ("c4_14b", 16, "host", "host"),
    ("c2_1p6b", 1, "device", "host"), ("c3_7b", 1, "device", "host"),
    # the set-up bench.py times by default: weights drawn and quantized on the device
    ("c4_14b", 16, "device", "device"), ("c3_7b", 8, "device", "device")])
def test_whole_step_at_benchmark_size_matches_oracle_on_sampled_products(name, batch, quantizer, weights):
    # quantizer = "device": the images come from rwkvq_quantize_dev, the oracle decodes the codes
    # unpacked from those images
    st = stack_mod.from_name(name, batch=batch, distinct_layers=2 if weights == "device" else 1, kmeans_iters=2,
                             quantizer=quantizer, weights=weights)
    _check_step(st, name)
    if weights == "device" and name == "c3_7b":      # the same images under another batch size
        st.set_batch(1)
        _check_step(st, name)


def _check_step(st, name):
    st.plan_step()
    for _ in range(2):                      # a second run must reproduce the first (outputs are cleared in the kernel)
        st.run_step()
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 0
    n = len(st.ops)
    picks = sorted({0, 1, 4, 5, 7, n // 2, n // 2 + 3, n - 8, n - 3, n - 1})
    kinds = set()
    for i in picks:
        op = st.ops[i]
        kinds.add((op.name, op.method))
        ref, tol = _oracle_product(st, op)
        y = op.y.double().cpu().numpy()
        assert np.isfinite(y).all()
        err = np.abs(y - ref)
        assert (err <= tol).all(), f"{name} op {i} ({op.name}, layer {op.layer}): max err/tol {float((err / tol).max())}"
    assert len(kinds) >= 4
    # every output of every product was written (none left at its cleared value by accident): spot-check norms
    for op in st.ops[:: max(1, n // 16)]:
        assert float(op.y.abs().sum()) > 0.0


@pytest.mark.parametrize("name,batch", [("c3_7b", 8), ("c3_7b", 1), ("c4_14b", 16)])
def test_host_buffer_step_overlaps_copies_without_changing_results(name, batch):
    """rwkvq_step_run_host at sizes where the activations arrive in chunks while the step runs and the
    outputs leave stage by stage: the host gets exactly what the device holds at the end of the step
    (no output copied before its stage was complete), and the step has read the NEW activations (none
    read before its chunk arrived): fresh inputs through the host path against the same inputs copied
    to the device first and a resident run."""
    st = stack_mod.from_name(name, batch=batch, distinct_layers=2, kmeans_iters=2, quantizer="device", weights="device")
    st.plan_step()
    st.run_step()
    torch.cuda.synchronize()
    g = torch.Generator().manual_seed(1234 + batch)
    halves = st.act_host.view(torch.float16)
    for rep in range(3):
        # new activations on the host only; the device arena keeps the old ones until the call copies them
        halves.copy_((torch.randn(halves.numel(), generator=g) * 0.5).to(torch.float16))
        st.y_host.zero_()
        st.run_step_host()
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        assert torch.equal(st.y_host, st.y_arena.cpu())
        assert torch.equal(st.act_arena.cpu(), st.act_host)
        y_host = st.y_host.view(torch.float32).clone()
        st.run_step()                       # resident run on the same (now copied) activations
        torch.cuda.synchronize()
        y_dev = st.y_arena.cpu().view(torch.float32)
        # the two runs differ only in the order of the fp32 reductions into y
        scale = float(y_dev.abs().max())
        assert float((y_host - y_dev).abs().max()) <= 1e-4 * scale
    op = st.ops[len(st.ops) // 2]
    ref, tol = _oracle_product(st, op)
    y = op.y.double().cpu().numpy()
    assert (np.abs(y - ref) <= tol).all()


def test_host_buffer_step_that_gives_up_releases_its_output_copies():
    """A host-buffer run whose stage barriers can never open (wait_skew) with a small poll limit: the
    kernel gives up by itself (ETIMEOUT), the output copies that were ordered behind the barriers are
    released all the same, the caller's synchronize returns, and the next run is correct again."""
    st = stack_mod.from_name("c3_7b", batch=8, distinct_layers=2, kmeans_iters=2, quantizer="device", weights="device")
    st.plan_step()
    st.run_step_host()
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 0
    good = st.y_host.clone()
    B.rwkvq_step_set_wait(st._plan, poll_limit=2000, wait_skew=1)
    st.run_step_host()
    torch.cuda.synchronize()
    assert B.rwkvq_device_status() == 8          # RWKVQ_ETIMEOUT; reading it clears the word
    B.rwkvq_step_set_wait(st._plan, poll_limit=0, wait_skew=0)
    for _ in range(2):
        st.y_host.zero_()
        st.run_step_host()
        torch.cuda.synchronize()
        assert B.rwkvq_device_status() == 0
        a, b = st.y_host.view(torch.float32), good.view(torch.float32)
        assert float((a - b).abs().max()) <= 1e-4 * float(b.abs().max())
