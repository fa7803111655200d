"""Shared helpers of the GPU parity tests: build logical codes with the oracle (or draw random
valid codes), pack them with the library, copy the image to the device."""
import numpy as np
import torch

from oracle import rwkvq_oracle as orc
from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import inputs


random_sq_codes = inputs.random_sq_codes
random_vq_codes = inputs.random_vq_codes
random_mu_codes = inputs.random_mu_codes


def decode(codes, method):
    """Oracle decode of logical codes -> float64 [oc, ic] (or [ic] for a vector)."""
    if method == B.RWKVQ_SQ:
        return orc.sq_decode(codes["q"], codes["scale"], codes["zero"])
    if codes["q"].ndim == 1:
        return orc.mu_decode(codes["codebook"], codes["q"])
    return orc.vq_decode(codes["codebook"], codes["q"])


class Packed:
    def __init__(self, codes, method, bits, oc, ic):
        self.codes, self.method, self.bits, self.oc, self.ic = codes, method, bits, oc, ic
        self.blob = B.rwkvq_pack(None, oc, ic, method, bits, codes=codes)
        self.desc = self.blob.desc
        self.dev = self.blob.to_device()
        self.w_hat = decode(codes, method)


def pack_sq(codes):
    oc, ic = codes["q"].shape
    return Packed(codes, B.RWKVQ_SQ, 3, oc, ic)


def pack_vq(codes, bits):
    oc, half = codes["q"].shape
    return Packed(codes, B.RWKVQ_VQ, bits, oc, half * 2)


def pack_mu(codes, bits=6):
    return Packed(codes, B.RWKVQ_VQ, bits, 1, codes["q"].shape[0] * 2)


def run_gemv(W: Packed, mu, x16, xp16, y_dtype=torch.float32):
    """x16, xp16: numpy float16 [B, ic].  Returns y as float64 numpy [B, oc]."""
    Bn = x16.shape[0]
    xd = torch.from_numpy(x16).cuda()
    xpd = torch.from_numpy(xp16).cuda() if mu is not None else None
    y = torch.full((Bn, W.oc), float("nan"), dtype=y_dtype, device="cuda")
    ws = torch.zeros(max(256, B.rwkvq_gemv_workspace_bytes(W.desc, Bn)), dtype=torch.uint8, device="cuda")
    args = (W.desc, W.dev, None if mu is None else mu.desc, None if mu is None else mu.dev, xd, xpd, Bn)
    B.rwkvq_gemv(*args, y, ws)
    y2 = torch.full_like(y, float("nan"))
    B.rwkvq_gemv(*args, y2, ws)          # the workspace is reusable without clearing
    torch.cuda.synchronize()
    assert torch.equal(y, y2), "second call on the same workspace differs"
    return y.double().cpu().numpy()


def reference(W: Packed, mu, x16, xp16):
    x = x16.astype(np.float64)
    xm = x if mu is None else orc.token_shift(x, xp16.astype(np.float64), mu.w_hat)
    return orc.gemv(W.w_hat, xm), orc.tolerance(W.w_hat, xm)
