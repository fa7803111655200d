"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module holds no quantization, decoding or multiplication arithmetic: it only
draws random numbers with the shapes and value distributions of the RWKV-6
projection workloads (Gaussian and heavy-tailed weight matrices, Gaussian
activations with a few amplified outlier channels, token-shift vectors in (0,1)).
Everything is returned as numpy arrays; fp16 data are numpy float16 arrays,
bf16 data are float32 arrays already rounded to bf16 precision plus their
uint16 bit patterns.
"""
from __future__ import annotations

import hashlib

import numpy as np

# Matrix set of one RWKV-6 block (time-mix R,K,V,G,O; channel-mix K,V,R) as
# (name, rows-as-multiple, cols-as-multiple, has_mu, stage).  "d" and "h" are
# replaced by the model width and the channel-mix hidden width.
LAYER_MATRICES = (
    ("tm_r", "d", "d", True, 0),
    ("tm_k", "d", "d", True, 0),
    ("tm_v", "d", "d", True, 0),
    ("tm_g", "d", "d", True, 0),
    ("tm_o", "d", "d", False, 1),
    ("cm_k", "h", "d", True, 2),
    ("cm_r", "d", "d", False, 2),
    ("cm_v", "d", "h", False, 3),
)

STACKS = {
    # name: (d, h, layers, vq_entries, batch sizes, outlier spec)
    "c2_1p6b": dict(d=2048, h=7168, layers=24, entries=64, batches=(1,), outliers=8),
    "c3_7b": dict(d=4096, h=14336, layers=32, entries=64, batches=(1, 8), outliers=8),
    "c4_14b": dict(d=4096, h=14336, layers=61, entries=256, batches=(16,), outliers=41),
}


def seed_of(*parts) -> int:
    """Stable 63-bit seed from a tuple of strings/ints (independent of PYTHONHASHSEED)."""
    h = hashlib.sha256("/".join(str(p) for p in parts).encode()).digest()
    return int.from_bytes(h[:8], "little") >> 1


def weight_kind(seed: int, heavy_fraction: float = 0.1) -> str:
    """Seeded coin: 'gauss' with probability 1-heavy_fraction, else 'student'."""
    u = np.random.default_rng(seed ^ 0x5EED).random()
    return "student" if u < heavy_fraction else "gauss"


def gen_weight(seed: int, oc: int, ic: int, kind: str = "gauss") -> np.ndarray:
    """fp16 weight matrix [oc, ic]: N(0, std 0.02) or Student-t(nu=3) * 0.01."""
    rng = np.random.default_rng(seed)
    if kind == "gauss":
        w = rng.standard_normal((oc, ic), dtype=np.float32) * np.float32(0.02)
    elif kind == "student":
        w = rng.standard_t(3.0, size=(oc, ic)).astype(np.float32) * np.float32(0.01)
    elif kind == "uniform":
        w = (rng.random((oc, ic), dtype=np.float32) - np.float32(0.5)) * np.float32(0.1)
    else:
        raise ValueError(kind)
    return w.astype(np.float16)


def gen_mu(seed: int, ic: int) -> np.ndarray:
    """fp16 token-shift vector of length ic, uniform in (0,1)."""
    rng = np.random.default_rng(seed)
    return rng.random(ic, dtype=np.float32).astype(np.float16)


def gen_activation(seed: int, batch: int, ic: int, n_outliers: int = 8, scale: float = 20.0):
    """fp32 activations [batch, ic]: N(0,1) with n_outliers seeded channels multiplied by
    `scale` (the same channels for every row).  Callers round to fp16 or bf16."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((batch, ic), dtype=np.float32)
    if n_outliers > 0:
        ch = rng.choice(ic, size=min(n_outliers, ic), replace=False)
        x[:, ch] *= np.float32(scale)
    return x


def outlier_channels(seed: int, ic: int, n_outliers: int) -> np.ndarray:
    """The channel set gen_activation amplifies for this seed (same draw order)."""
    rng = np.random.default_rng(seed)
    return rng.choice(ic, size=min(n_outliers, ic), replace=False)


def gen_activation_pair(seed: int, batch: int, ic: int, n_outliers: int = 8, scale: float = 20.0):
    """(x, x_prev) fp32 pair sharing one outlier-channel set."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((batch, ic), dtype=np.float32)
    xp = rng.standard_normal((batch, ic), dtype=np.float32)
    if n_outliers > 0:
        ch = rng.choice(ic, size=min(n_outliers, ic), replace=False)
        x[:, ch] *= np.float32(scale)
        xp[:, ch] *= np.float32(scale)
    return x, xp


def random_sq_codes(seed: int, oc: int, ic: int, group: int = 128, bits: int = 3) -> dict:
    """Valid logical SQ codes drawn at random (no quantizer involved): codes uniform in
    [0, 2^bits), fp16 scales in [0.005, 0.025), integer zero points in [0, 2^bits)."""
    rng = np.random.default_rng(seed)
    q = rng.integers(0, 1 << bits, size=(oc, ic), dtype=np.uint8)
    s = (rng.random((oc, ic // group)) * 0.02 + 0.005).astype(np.float16)
    z = rng.integers(0, 1 << bits, size=(oc, ic // group)).astype(np.float16)
    return dict(q=q, scale=s, zero=z)


def random_vq_codes(seed: int, oc: int, ic: int, bits: int, tile: int = 256) -> dict:
    """Valid logical VQ codes drawn at random: indices uniform in [0, 2^bits), one fp16 codebook
    of N(0, 0.02) 2-vectors per tile x tile block."""
    rng = np.random.default_rng(seed)
    E = 1 << bits
    idx = rng.integers(0, E, size=(oc, ic // 2), dtype=np.uint8)
    cb = (rng.standard_normal((oc // tile, ic // tile, E, 2)) * 0.02).astype(np.float16)
    return dict(q=idx, codebook=cb)


def random_mu_codes(seed: int, ic: int, bits: int = 6) -> dict:
    """Valid logical codes of a token-shift vector: indices uniform, codebook uniform in (0,1)."""
    rng = np.random.default_rng(seed)
    E = 1 << bits
    return dict(q=rng.integers(0, E, size=(ic // 2,), dtype=np.uint8),
                codebook=rng.random((E, 2)).astype(np.float16))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even) and return the uint16 bit patterns.
    Pure number-format conversion (no method arithmetic)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def layer_shapes(d: int, h: int):
    """[(name, oc, ic, has_mu, stage)] for one block."""
    dim = {"d": d, "h": h}
    return [(n, dim[r], dim[c], m, s) for (n, r, c, m, s) in LAYER_MATRICES]
