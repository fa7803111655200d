"""Synthetic RWKV-6-shaped projection stacks: seeded weights -> proxy selection -> packed images on
the device, plus the activation buffers of one decode step.

Only marshalling lives here: the selection runs in rwkvq_proxy_select, quantization and packing in
rwkvq_pack (or, with quantizer="device", in rwkvq_quantize_dev), the products in rwkvq_gemv /
rwkvq_step_run.
"""
from __future__ import annotations

import math
import time

import numpy as np
import torch

from . import binding as B
from . import inputs


class MatrixEntry:
    __slots__ = ("layer", "name", "oc", "ic", "kind", "seed", "stage", "has_mu", "method", "pc", "pf",
                 "desc", "image", "mu_desc", "mu_image", "x", "xprev", "y", "act_off")


class _DeviceBlob:
    """A matrix quantized and packed by rwkvq_quantize_dev: same surface as binding.Blob."""

    def __init__(self, desc, image):
        self.desc, self._image = desc, image

    def to_device(self, device="cuda"):
        return self._image.clone()

    def export_codes(self):
        return B.rwkvq_image_unpack(self._image.cpu().numpy())[1]


def _device_blob(w_dev, oc, ic, method, bits, kmeans_iters, seed):
    d = B.rwkvq_desc_for(oc, ic, method, bits)
    image = torch.empty(int(d.image_bytes), dtype=torch.uint8, device=w_dev.device)
    ws = torch.empty(B.rwkvq_quantize_workspace_bytes(), dtype=torch.uint8, device=w_dev.device)
    d = B.rwkvq_quantize_dev(w_dev, oc, ic, method, bits, image, ws, kmeans_iters=kmeans_iters, seed=seed)
    return _DeviceBlob(d, image)


def gen_weight_device(seed: int, oc: int, ic: int, kind: str, device="cuda"):
    """fp16 weight matrix [oc, ic] drawn on the device from a seeded generator: N(0, std 0.02), or
    Student-t(nu=3) * 0.01 as a normal variate over the root of a chi-square(3) variate / 3.  Same
    distributions as inputs.gen_weight, other values: set-up of the large stacks without the host
    generator's minutes."""
    gen = torch.Generator(device=device).manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    z = torch.randn((oc, ic), generator=gen, device=device, dtype=torch.float32)
    if kind == "gauss":
        return (z * 0.02).to(torch.float16)
    if kind != "student":
        raise ValueError(kind)
    chi = torch.zeros_like(z)
    for _ in range(3):
        n = torch.randn((oc, ic), generator=gen, device=device, dtype=torch.float32)
        chi.addcmul_(n, n)
    return (z * torch.rsqrt(chi / 3.0) * 0.01).to(torch.float16)


class Stack:
    """All projection matrices of `layers` RWKV-6 blocks of width d and channel-mix width h.

    Per matrix the weight distribution is N(0, 0.02) or Student-t(3)*0.01 by a seeded coin; the
    SQ/VQ method comes from rwkvq_proxy_select with tau_c at the widest gap of the measured P_c
    (rwkvq_tau_largest_gap) and tau_f = +inf; SQ is 3-bit group-128, VQ uses 2-D vectors with
    `entries` codebook entries per 256x256 tile.  The four time-mix input projections and the
    channel-mix key projection get a VQ-coded token-shift vector.  `distinct_layers` > 0 draws
    weights for that many layers only and reuses their values (in separate device buffers) for the
    remaining layers.  weights="device" draws the weights with a seeded generator on the device
    (quantizer="device" only); weights="host" uses the numpy generators of the inputs module.
    """

    def __init__(self, d: int, h: int, layers: int, entries: int, batch: int, n_outliers: int = 8,
                 heavy_fraction: float = 0.1, tag: str = "stack", device: str = "cuda",
                 distinct_layers: int = 0, force_method: int | None = None, kmeans_iters: int = 10,
                 verbose: bool = False, quantizer: str = "host", weights: str = "host"):
        assert quantizer in ("host", "device") and weights in ("host", "device")
        if weights == "device" and quantizer != "device":
            raise ValueError("weights drawn on the device are quantized on the device")
        self.quantizer, self.weights = quantizer, weights
        self.d, self.h, self.layers, self.entries = d, h, layers, entries
        self.n_outliers = n_outliers
        self.tag, self.device = tag, device
        self.vq_bits = 6 if entries == 64 else 8
        self.ops: list[MatrixEntry] = []
        self.setup_seconds = {}
        t0 = time.time()
        shapes = inputs.layer_shapes(d, h)
        self.shapes = shapes
        n_src = layers if distinct_layers <= 0 else min(layers, distinct_layers)
        self.n_src = n_src
        # pass 1: weights of the source layers, P_c / P_f on the device
        src_w = {}
        for l in range(n_src):
            mats = []
            for (name, oc, ic, has_mu, stage) in shapes:
                seed = inputs.seed_of(tag, l, name)
                kind = inputs.weight_kind(seed, heavy_fraction)
                if weights == "device":
                    w_dev = gen_weight_device(seed, oc, ic, kind, device)
                    src_w[(l, name)] = (w_dev, kind, seed)
                else:
                    w = inputs.gen_weight(seed, oc, ic, kind)
                    w_dev = torch.from_numpy(w).to(device)
                    src_w[(l, name)] = (w, kind, seed)
                mats.append(w_dev)
            ws = torch.empty(B.rwkvq_proxy_workspace_bytes(len(mats)), dtype=torch.uint8, device=device)
            pc, pf, _ = B.rwkvq_proxy_select(mats, 4, math.inf, math.inf, ws)
            for (name, *_), a, b in zip(shapes, pc, pf):
                src_w[(l, name)] += (float(a), float(b))
            del mats, ws
        self.setup_seconds["generate+proxy"] = time.time() - t0
        t0 = time.time()
        all_pc = np.array([v[3] for v in src_w.values()])
        self.tau_c = B.rwkvq_tau_largest_gap(all_pc)
        self.tau_f = math.inf
        # pass 2: selection (Eq. 18 inside the library), quantize + pack, upload
        packed = {}
        for l in range(n_src):
            mats = [src_w[(l, name)][0] if weights == "device" else torch.from_numpy(src_w[(l, name)][0]).to(device)
                    for (name, *_r) in shapes]
            ws = torch.empty(B.rwkvq_proxy_workspace_bytes(len(mats)), dtype=torch.uint8, device=device)
            _, _, phi = B.rwkvq_proxy_select(mats, 4, self.tau_c, self.tau_f, ws)
            del ws
            for (name, oc, ic, has_mu, stage), p, w_dev in zip(shapes, phi, mats):
                w, kind, seed, pc_v, pf_v = src_w[(l, name)]
                method = int(p) if force_method is None else force_method
                if quantizer == "device":
                    bits = 3 if method == B.RWKVQ_SQ else self.vq_bits
                    blob = _device_blob(w_dev, oc, ic, method, bits, kmeans_iters, seed)
                elif method == B.RWKVQ_SQ:
                    blob = B.rwkvq_pack(w, oc, ic, B.RWKVQ_SQ, 3)
                else:
                    blob = B.rwkvq_pack(w, oc, ic, B.RWKVQ_VQ, self.vq_bits, kmeans_iters=kmeans_iters, seed=seed)
                mu_blob = None
                if has_mu and quantizer == "device":
                    mu = torch.from_numpy(inputs.gen_mu(seed ^ 0xABCD, ic)).to(device)
                    mu_blob = _device_blob(mu, 1, ic, B.RWKVQ_VQ, self.vq_bits, kmeans_iters, seed + 1)
                elif has_mu:
                    mu = inputs.gen_mu(seed ^ 0xABCD, ic)
                    mu_blob = B.rwkvq_pack(mu.reshape(1, -1), 1, ic, B.RWKVQ_VQ, self.vq_bits,
                                           kmeans_iters=kmeans_iters, seed=seed + 1)
                packed[(l, name)] = (blob, mu_blob, kind, seed, method, pc_v, pf_v)
                if verbose:
                    print(f"layer {l} {name}: {kind} pc={pc_v:.3f} -> {'SQ' if method else 'VQ'}", flush=True)
            del mats
            for (name, *_r) in shapes:
                src_w.pop((l, name))
        self.setup_seconds["select+pack"] = time.time() - t0
        t0 = time.time()
        self._packed = packed  # keeps the blobs (logical codes on request) for parity checks
        # one device image per (layer, matrix): layers beyond the source layers get copies of their own
        self._images = {}
        for l in range(layers):
            for (name, oc, ic, has_mu, stage) in shapes:
                blob, mu_blob, *_r = packed[(l % n_src, name)]
                if l < n_src and isinstance(blob, _DeviceBlob):      # already on the device: no second copy
                    self._images[(l, name)] = (blob._image, mu_blob._image if has_mu else None)
                else:
                    self._images[(l, name)] = (blob.to_device(device), mu_blob.to_device(device) if has_mu else None)
        self.setup_seconds["upload"] = time.time() - t0
        self.set_batch(batch)

    def set_batch(self, batch: int):
        """(Re)builds the activation and output arenas and the product list for a decode batch; the
        packed images stay where they are."""
        t0 = time.time()
        device, shapes, layers = self.device, self.shapes, self.layers
        self.batch = batch
        self.ops = []
        if getattr(self, "_plan", None) is not None:
            B.rwkvq_step_plan_release(self._plan)
        self._plan = None
        # Activations of every product live in one device arena and the outputs in another, so a
        # step's inputs arrive in one host-to-device copy and its results leave in one copy back.
        def _al(n):
            return (n + 255) // 256 * 256
        act_off, y_off, slots = 0, 0, []
        for l in range(layers):
            for (name, oc, ic, has_mu, stage) in shapes:
                xo = act_off
                act_off += _al(batch * ic * 2)
                po = None
                if has_mu:
                    po = act_off
                    act_off += _al(batch * ic * 2)
                slots.append((xo, po, y_off))
                y_off += _al(batch * oc * 4)
        self.act_host = torch.empty(act_off, dtype=torch.uint8).pin_memory() if device != "cpu" else torch.empty(act_off, dtype=torch.uint8)
        self.act_arena = torch.empty(act_off, dtype=torch.uint8, device=device)
        self.y_arena = torch.zeros(y_off, dtype=torch.uint8, device=device)
        self.y_host = torch.empty(y_off, dtype=torch.uint8).pin_memory() if device != "cpu" else torch.empty(y_off, dtype=torch.uint8)
        act_np = self.act_host.numpy()
        k = 0
        for l in range(layers):
            src = l % self.n_src
            for (name, oc, ic, has_mu, stage) in shapes:
                blob, mu_blob, kind, seed, method, pc_v, pf_v = self._packed[(src, name)]
                xo, po, yo = slots[k]
                k += 1
                e = MatrixEntry()
                e.layer, e.name, e.oc, e.ic, e.kind, e.seed = l, name, oc, ic, kind, seed
                e.stage, e.has_mu, e.method, e.pc, e.pf = 4 * l + stage, has_mu, method, pc_v, pf_v
                e.desc, e.image = blob.desc, self._images[(l, name)][0]
                e.mu_desc, e.mu_image = (mu_blob.desc, self._images[(l, name)][1]) if has_mu else (None, None)
                act_seed = inputs.seed_of(self.tag, "act", l, name)
                nb = batch * ic * 2
                if has_mu:
                    x, xp = inputs.gen_activation_pair(act_seed, batch, ic, self.n_outliers)
                    act_np[po:po + nb] = xp.astype(np.float16).reshape(-1).view(np.uint8)
                    e.xprev = self.act_arena[po:po + nb].view(torch.float16).view(batch, ic)
                else:
                    x = inputs.gen_activation(act_seed, batch, ic, self.n_outliers)
                    e.xprev = None
                act_np[xo:xo + nb] = x.astype(np.float16).reshape(-1).view(np.uint8)
                e.x = self.act_arena[xo:xo + nb].view(torch.float16).view(batch, ic)
                e.y = self.y_arena[yo:yo + batch * oc * 4].view(torch.float32).view(batch, oc)
                e.act_off = (xo, po, yo)
                self.ops.append(e)
        self.act_arena.copy_(self.act_host)
        self.ops.sort(key=lambda o: o.stage)
        self.n_weights = sum(o.oc * o.ic for o in self.ops)
        self.stream_bytes = sum(int(o.desc.stream_bytes) + (int(o.mu_desc.stream_bytes) if o.has_mu else 0)
                                for o in self.ops)
        self.act_bytes = sum(batch * o.ic * 2 * (2 if o.has_mu else 1) + batch * o.oc * 4 for o in self.ops)
        self.n_sq = sum(1 for o in self.ops if o.method == B.RWKVQ_SQ)
        self.n_stages = len({o.stage for o in self.ops})
        ws_bytes = max(B.rwkvq_gemv_workspace_bytes(o.desc, batch) for o in self.ops)
        self.workspace = torch.zeros(max(ws_bytes, 256), dtype=torch.uint8, device=device)
        self.setup_seconds["activations"] = time.time() - t0

    def host_codes(self, op: MatrixEntry):
        """Logical codes (numpy) of a matrix and of its mu vector, exported by the packer."""
        blob, mu_blob, *_ = self._packed[(op.layer % self.n_src, op.name)]
        return blob.export_codes(), (mu_blob.export_codes() if mu_blob is not None else None)

    # ---- one decode step ----------------------------------------------------------------------
    def run_ops(self, stream=None):
        """One rwkvq_gemv launch per product, in stage order."""
        for o in self.ops:
            B.rwkvq_gemv(o.desc, o.image, o.mu_desc, o.mu_image, o.x, o.xprev, self.batch, o.y,
                         self.workspace, stream)
        return len(self.ops)

    def plan_step(self):
        entries = [dict(desc=o.desc, W=o.image, mu_desc=o.mu_desc, mu=o.mu_image, x=o.x, xprev=o.xprev,
                        y=o.y, stage=o.stage) for o in self.ops]
        ops = B.make_ops(entries)
        nbytes = B.rwkvq_step_plan_bytes(ops, self.batch)
        if nbytes == 0:
            raise RuntimeError("rwkvq_step_plan_bytes returned 0 (plan rejected)")
        self._plan = torch.zeros(nbytes, dtype=torch.uint8, device=self.device)
        B.rwkvq_step_plan(ops, self.batch, self._plan)
        torch.cuda.synchronize()

    def run_step(self, stream=None):
        """The whole step as one persistent launch (rwkvq_step_run)."""
        if self._plan is None:
            self.plan_step()
        B.rwkvq_step_run(self._plan, stream)
        return 1

    def run_step_host(self, stream=None):
        """The step with its activations read from and its outputs written to pinned host memory
        (rwkvq_step_run_host); the caller synchronizes before reading self.y_host."""
        if self._plan is None:
            self.plan_step()
        B.rwkvq_step_run_host(self._plan, self.act_host, self.act_arena, self.y_arena, self.y_host, stream)
        return 1


def from_name(name: str, batch: int | None = None, **kw) -> Stack:
    spec = inputs.STACKS[name]
    b = spec["batches"][0] if batch is None else batch
    return Stack(spec["d"], spec["h"], kw.pop("layers", spec["layers"]), spec["entries"], b,
                 n_outliers=spec["outliers"], tag=name, **kw)


class BlockOp:
    __slots__ = ("layer", "name", "oc", "ic", "method", "desc", "image", "mu_desc", "mu_image", "y", "stage", "xform",
                 "x", "xprev", "blob", "mu_blob")


class BlockStack:
    """`layers` RWKV blocks as Appendix A.1 writes them, chained: per block the time-mixing projections R, K,
    V (token-shift mix each), the WKV recurrence and sigmoid gate in front of O (Eqs. 23-24), the channel-mixing
    projections cm_k and cm_r (token-shift mix each, input = O's output), the squared ReLU in front of cm_v
    (Eq. 27); the next block's input is sigmoid(cm_r) * cm_v.  Every element-wise operator runs inside the
    persistent decode step (rwkvq_input_xform), so the four stages of a block are real data dependencies.
    The paper's block has no gate matrix and prints neither norms nor residual connections: none here.
    Without a normalisation the squared ReLU makes the activations of a chain of blocks collapse to zero
    or overflow within a few blocks (measured: zero by the third block, or NaN by the eighth), so the
    inputs of time mixing (from the second block on) and of channel mixing are divided by their root
    mean square (RWKVQ_INF_RMSNORM), the places where the models the paper quantizes normalise.
    Weights, method selection and quantization as in Stack (drawn and quantized on the device)."""

    def __init__(self, d: int, h: int, layers: int, entries: int, batch: int, n_outliers: int = 8,
                 heavy_fraction: float = 0.1, tag: str = "block", device: str = "cuda", kmeans_iters: int = 10,
                 weight_scale: float = 1.0):
        self.d, self.h, self.layers, self.batch, self.device, self.tag = d, h, layers, batch, device, tag
        self.n_outliers = n_outliers
        vq_bits = 6 if entries == 64 else 8
        names = (("R", d, d, True, 0), ("K", d, d, True, 0), ("V", d, d, True, 0), ("O", d, d, False, 1),
                 ("cm_k", h, d, True, 2), ("cm_r", d, d, True, 2), ("cm_v", d, h, False, 3))
        t0 = time.time()
        raw, pcs = {}, []
        for l in range(layers):
            mats = []
            for (name, oc, ic, has_mu, stage) in names:
                seed = inputs.seed_of(tag, l, name)
                kind = inputs.weight_kind(seed, heavy_fraction)
                w = gen_weight_device(seed, oc, ic, kind, device)
                if weight_scale != 1.0:
                    w = (w.float() * weight_scale).to(torch.float16)
                raw[(l, name)] = (w, seed)
                mats.append(w)
            ws = torch.empty(B.rwkvq_proxy_workspace_bytes(len(mats)), dtype=torch.uint8, device=device)
            pc, _, _ = B.rwkvq_proxy_select(mats, 4, math.inf, math.inf, ws)
            pcs.extend(float(v) for v in pc)
        self.tau_c = B.rwkvq_tau_largest_gap(np.array(pcs))
        z32 = lambda *s: torch.zeros(s, dtype=torch.float32, device=device)
        z16 = lambda *s: torch.zeros(s, dtype=torch.float16, device=device)
        self.x0 = z16(batch, d)
        self.x0_host = torch.zeros((batch, d), dtype=torch.float16).pin_memory()
        self.ops: list[BlockOp] = []
        self.states = []
        gen = torch.Generator(device=device).manual_seed(inputs.seed_of(tag, "wkv") & 0x7FFFFFFF)
        prev = None
        k = 0
        for l in range(layers):
            ws = torch.empty(B.rwkvq_proxy_workspace_bytes(len(names)), dtype=torch.uint8, device=device)
            _, _, phi = B.rwkvq_proxy_select([raw[(l, n[0])][0] for n in names], 4, self.tau_c, math.inf, ws)
            y = {}
            st = dict(a=z32(batch, d), b=z32(batch, d), p=torch.full((batch, d), -1e30, dtype=torch.float32, device=device),
                      u=torch.randn(d, generator=gen, device=device) * 0.3,
                      w=torch.rand(d, generator=gen, device=device) * 0.95 + 0.05)
            self.states.append(st)
            layer_ops = {}
            for (name, oc, ic, has_mu, stage), p in zip(names, phi):
                w, seed = raw.pop((l, name))
                method = int(p)
                blob = _device_blob(w, oc, ic, method, 3 if method == B.RWKVQ_SQ else vq_bits, kmeans_iters, seed)
                o = BlockOp()
                o.layer, o.name, o.oc, o.ic, o.method, o.blob = l, name, oc, ic, method, blob
                o.desc, o.image = blob.desc, blob._image
                o.mu_desc = o.mu_image = o.mu_blob = o.xprev = o.x = None
                if has_mu:
                    mu = torch.from_numpy(inputs.gen_mu(seed ^ 0xABCD, ic)).to(device)
                    o.mu_blob = _device_blob(mu, 1, ic, B.RWKVQ_VQ, vq_bits, kmeans_iters, seed + 1)
                    o.mu_desc, o.mu_image = o.mu_blob.desc, o.mu_blob._image
                    o.xprev = z16(batch, ic)                 # this product's previous-token input, advanced by the step
                o.y = z32(batch, oc)
                o.stage = 4 * l + stage
                y[name] = o.y
                layer_ops[name] = o
                self.ops.append(o)
                k += 1
            for name in ("R", "K", "V"):
                o = layer_ops[name]
                if prev is None:
                    o.x, o.xform = self.x0, dict(kind=B.RWKVQ_IN_BUFFER, xprev_out=o.xprev)
                else:
                    o.xform = dict(kind=B.RWKVQ_IN_F32, src=prev[1], gate=prev[0], xprev_out=o.xprev, rmsnorm=True)
            layer_ops["O"].xform = dict(kind=B.RWKVQ_IN_WKV, src=y["R"], k=y["K"], v=y["V"], state_a=st["a"], state_b=st["b"],
                                        state_p=st["p"], u=st["u"], w=st["w"])
            for name in ("cm_k", "cm_r"):
                layer_ops[name].xform = dict(kind=B.RWKVQ_IN_F32, src=y["O"], xprev_out=layer_ops[name].xprev, rmsnorm=True)
            layer_ops["cm_v"].xform = dict(kind=B.RWKVQ_IN_RELU2, src=y["cm_k"])
            prev = (y["cm_r"], y["cm_v"])
        self.out_r, self.out_v = prev
        self.out_host = torch.zeros((2, batch, d), dtype=torch.float32).pin_memory()
        self.ops.sort(key=lambda o: o.stage)
        self.n_weights = sum(o.oc * o.ic for o in self.ops)
        self.stream_bytes = sum(int(o.desc.stream_bytes) + (int(o.mu_desc.stream_bytes) if o.mu_desc is not None else 0)
                                for o in self.ops)
        # fp32 outputs written once and read once or twice by the next stage, fp16 previous-token states, WKV state
        self.act_bytes = (sum(batch * o.oc * 4 * 2 + (batch * o.ic * 2 * 2 if o.xprev is not None else 0) for o in self.ops)
                          + layers * batch * d * 4 * 6)
        self.n_sq = sum(1 for o in self.ops if o.method == B.RWKVQ_SQ)
        self.n_stages = 4 * layers
        self.setup_s = time.time() - t0
        entries_ = [dict(desc=o.desc, W=o.image, mu_desc=o.mu_desc, mu=o.mu_image, x=o.x, xprev=o.xprev, y=o.y, stage=o.stage,
                         **{"in": o.xform}) for o in self.ops]
        ops_arr = B.make_ops(entries_)
        nbytes = B.rwkvq_step_plan_bytes(ops_arr, batch)
        if nbytes == 0:
            raise RuntimeError("rwkvq_step_plan_bytes returned 0 (plan rejected)")
        self._plan = torch.zeros(nbytes, dtype=torch.uint8, device=device)
        B.rwkvq_step_plan(ops_arr, batch, self._plan)
        torch.cuda.synchronize()

    def reset_state(self):
        """Start of a sequence: empty WKV history, zero previous-token inputs."""
        for st in self.states:
            st["a"].zero_(); st["b"].zero_(); st["p"].fill_(-1e30)
        for o in self.ops:
            if o.xprev is not None:
                o.xprev.zero_()

    def set_token(self, seed: int):
        """A fresh seeded token (fp16 activations with outlier channels) in the pinned host buffer."""
        self.x0_host.copy_(torch.from_numpy(inputs.gen_activation(seed, self.batch, self.d, self.n_outliers).astype(np.float16)))

    def run_step(self, stream=None):
        """One token through every block: one persistent launch; the input is whatever x0 holds."""
        B.rwkvq_step_run(self._plan, stream)

    def run_step_host(self, stream=None):
        """The token comes from pinned host memory and the last block's cm_r / cm_v outputs (whose gated
        product is the model's hidden state, Eq. 27) go back to it; the caller synchronizes."""
        self.x0.copy_(self.x0_host, non_blocking=True)
        B.rwkvq_step_run(self._plan, stream)
        self.out_host[0].copy_(self.out_r, non_blocking=True)
        self.out_host[1].copy_(self.out_v, non_blocking=True)

    def host_codes(self, op: BlockOp):
        return op.blob.export_codes(), (op.mu_blob.export_codes() if op.mu_blob is not None else None)
