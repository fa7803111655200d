"""rwkvq_gemv_static -- the decode product for callers that may not allocate device memory (the
scratch is an array inside the library) -- must give what rwkvq_gemv gives with a caller-owned
workspace, bit for bit (the partial sums are combined in the same fixed order), and both must match
the oracle.  Collected last on purpose: a failure here stops nothing else."""
import numpy as np
import pytest
import torch

from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _both(W, mu, x16, xp16):
    Bn = x16.shape[0]
    xd = torch.from_numpy(x16).cuda()
    xpd = torch.from_numpy(xp16).cuda() if mu is not None else None
    args = (W.desc, W.dev, None if mu is None else mu.desc, None if mu is None else mu.dev, xd, xpd, Bn)
    y_ref = torch.full((Bn, W.oc), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.zeros(max(256, B.rwkvq_gemv_workspace_bytes(W.desc, Bn)), dtype=torch.uint8, device="cuda")
    B.rwkvq_gemv(*args, y_ref, ws)
    outs = []
    for _ in range(2):          # two calls in a row share the library's scratch array
        y = torch.full_like(y_ref, float("nan"))
        B.rwkvq_gemv_static(*args, y)
        outs.append(y)
    torch.cuda.synchronize()
    return y_ref.double().cpu().numpy(), [o.double().cpu().numpy() for o in outs]


@pytest.mark.parametrize("fmt,oc,ic,Bn", [("sq", 2048, 2048, 1), ("sq", 256, 7168, 8), ("vq", 512, 4096, 16), ("sq", 128, 256, 3)])
def test_static_scratch_variant_matches_workspace_variant(fmt, oc, ic, Bn):
    W = H.pack_sq(H.random_sq_codes(oc + ic, oc, ic)) if fmt == "sq" else H.pack_vq(H.random_vq_codes(oc + ic, oc, ic, 6), 6)
    mu = H.pack_mu(H.random_mu_codes(ic, ic)) if Bn != 3 else None
    x, xp = inputs.gen_activation_pair(Bn + ic, Bn, ic, n_outliers=8)
    x16, xp16 = x.astype(np.float16), xp.astype(np.float16)
    y_ws, ys = _both(W, mu, x16, xp16)
    ref, tol = H.reference(W, mu, x16, xp16)          # the oracle's fp64 product and the stated tolerance
    assert (np.abs(y_ws - ref) <= tol).all()
    for y in ys:
        assert np.isfinite(y).all()
        assert (np.abs(y - ref) <= tol).all()
        assert np.array_equal(y, y_ws)
    assert B.rwkvq_device_status() == 0


def test_static_scratch_variant_refuses_products_beyond_its_array():
    assert B.rwkvq_gemv_static_max_scratch_bytes() == 8 << 20
    # a product whose split-K scratch exceeds the built-in array (checked from the sizes alone, before any launch)
    oc, ic, Bn = 57344, 256 * 40, 16
    d = B.Desc(method=B.RWKVQ_VQ, bits=6, oc=oc, ic=ic, group=0, vec_dim=2, tile=256, entries=64, oc_pad=oc, ic_pad=ic,
               image_bytes=0, stream_bytes=0)
    need = B.rwkvq_gemv_workspace_bytes(d, Bn)
    if need <= B.rwkvq_gemv_static_max_scratch_bytes():
        pytest.skip("no shape in range exceeds the array")
    dummy = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.RwkvqError) as e:
        B.rwkvq_gemv_static(d, dummy, None, None, dummy, None, Bn, dummy)
    assert e.value.status == 5
