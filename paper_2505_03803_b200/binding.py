"""Thin ctypes binding of librwkvq.so: argument marshalling only.

Names mirror the C ABI in include/rwkvq.h.  Device memory and streams come from
PyTorch (torch.Tensor.data_ptr(), torch.cuda.current_stream()); every step of the
path runs inside the library's kernels.  There is no CPU fallback: if the shared
library is missing this module raises at first use.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librwkvq.so")

RWKVQ_VQ, RWKVQ_SQ = 0, 1
RWKVQ_F32, RWKVQ_F16, RWKVQ_BF16 = 0, 1, 2
STATUS_NAMES = ["OK", "EINVAL", "ESHAPE", "EALIGN", "ENONFINITE", "ENOMEM", "ECUDA", "EUNSUPPORTED", "ETIMEOUT"]


class RwkvqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        msg = lib().rwkvq_status_str(status).decode()
        extra = ""
        if status == 6:
            extra = ": " + lib().rwkvq_last_cuda_error().decode()
        super().__init__(f"{where}: RWKVQ_{name} ({msg}{extra})")


class Codes(C.Structure):
    _fields_ = [("q", C.c_void_p), ("scale", C.c_void_p), ("zero", C.c_void_p), ("codebook", C.c_void_p)]


class QuantCfg(C.Structure):
    _fields_ = [("method", C.c_int32), ("bits", C.c_int32), ("group", C.c_int32), ("vec_dim", C.c_int32),
                ("tile", C.c_int32), ("kmeans_iters", C.c_int32), ("seed", C.c_uint64),
                ("codes_in", C.POINTER(Codes))]


class Desc(C.Structure):
    _fields_ = [("method", C.c_int32), ("bits", C.c_int32), ("oc", C.c_int32), ("ic", C.c_int32),
                ("group", C.c_int32), ("vec_dim", C.c_int32), ("tile", C.c_int32), ("entries", C.c_int32),
                ("oc_pad", C.c_int32), ("ic_pad", C.c_int32), ("image_bytes", C.c_uint64),
                ("stream_bytes", C.c_uint64)]


RWKVQ_IN_BUFFER, RWKVQ_IN_WKV, RWKVQ_IN_RELU2, RWKVQ_IN_F32 = 0, 1, 2, 3
RWKVQ_INF_RMSNORM = 1


class InputXform(C.Structure):
    _fields_ = [("kind", C.c_int32), ("flags", C.c_int32), ("src_f32", C.c_void_p), ("k_f32", C.c_void_p),
                ("v_f32", C.c_void_p), ("state_a", C.c_void_p), ("state_b", C.c_void_p), ("state_p", C.c_void_p),
                ("u_f32", C.c_void_p), ("w_f32", C.c_void_p), ("gate_f32", C.c_void_p), ("xprev_out_fp16", C.c_void_p), ("scale_f32", C.c_void_p)]


class GemvOp(C.Structure):
    _fields_ = [("W_desc", Desc), ("W_image_dev", C.c_void_p), ("mu_desc", Desc), ("mu_image_dev", C.c_void_p),
                ("x_fp16_dev", C.c_void_p), ("xprev_fp16_dev", C.c_void_p), ("y_dev", C.c_void_p),
                ("stage", C.c_int32), ("y_dtype", C.c_int32), ("in_", InputXform)]


class PrefillOp(C.Structure):
    _fields_ = [("W_desc", C.POINTER(Desc)), ("W_image_dev", C.c_void_p), ("mu_desc", C.POINTER(Desc)),
                ("mu_image_dev", C.c_void_p), ("X_bf16_dev", C.c_void_p), ("xprev0_bf16_dev", C.c_void_p),
                ("Y_dev", C.c_void_p), ("workspace_dev", C.c_void_p), ("workspace_bytes", C.c_size_t)]


EXPORTS = [
    "rwkvq_pack", "rwkvq_blob_desc", "rwkvq_blob_nbytes", "rwkvq_blob_image", "rwkvq_blob_export_codes",
    "rwkvq_image_unpack", "rwkvq_blob_free", "rwkvq_proxy_workspace_bytes", "rwkvq_proxy_select",
    "rwkvq_gemv_workspace_bytes", "rwkvq_gemv", "rwkvq_gemv_static", "rwkvq_gemv_static_max_scratch_bytes", "rwkvq_step_plan_bytes", "rwkvq_step_plan", "rwkvq_step_run",
    "rwkvq_step_run_host", "rwkvq_step_plan_release", "rwkvq_step_set_wait", "rwkvq_step_plan_cover",
    "rwkvq_prefill_workspace_bytes", "rwkvq_gemm_prefill", "rwkvq_gemm_prefill_grouped", "rwkvq_dequant", "rwkvq_device_status",
    "rwkvq_status_str", "rwkvq_last_cuda_error",
    "rwkvq_proxy_family", "rwkvq_proxy_select_bf16", "rwkvq_proxy_f32_workspace_bytes", "rwkvq_proxy_select_f32",
    "rwkvq_proxy_segments_workspace_bytes", "rwkvq_proxy_segments", "rwkvq_tau_for_fraction", "rwkvq_tau_largest_gap", "rwkvq_quant_error_workspace_bytes", "rwkvq_quant_error",
    "rwkvq_desc_for", "rwkvq_quantize_workspace_bytes", "rwkvq_quantize_dev", "rwkvq_calib_representative",
    "rwkvq_quantize_dev_async", "rwkvq_quantize_check",
]

_lib = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2505_03803_b200.build` "
            "(needs nvcc); this package has no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp, i32, sz, dbl = C.c_void_p, C.c_int, C.c_size_t, C.c_double
    L.rwkvq_pack.argtypes = [vp, i32, i32, C.POINTER(QuantCfg), C.POINTER(vp)]
    L.rwkvq_blob_desc.argtypes = [vp, C.POINTER(Desc)]
    L.rwkvq_blob_nbytes.argtypes = [vp]
    L.rwkvq_blob_nbytes.restype = sz
    L.rwkvq_blob_image.argtypes = [vp, vp, sz]
    L.rwkvq_blob_export_codes.argtypes = [vp, C.POINTER(Codes)]
    L.rwkvq_image_unpack.argtypes = [vp, sz, C.POINTER(Desc), C.POINTER(Codes)]
    L.rwkvq_blob_free.argtypes = [vp]
    L.rwkvq_blob_free.restype = None
    L.rwkvq_status_str.argtypes = [i32]
    L.rwkvq_status_str.restype = C.c_char_p
    L.rwkvq_last_cuda_error.restype = C.c_char_p
    if hasattr(L, "rwkvq_gemv"):
        L.rwkvq_gemv_workspace_bytes.argtypes = [C.POINTER(Desc), i32]
        L.rwkvq_gemv_workspace_bytes.restype = sz
        L.rwkvq_gemv.argtypes = [C.POINTER(Desc), vp, C.POINTER(Desc), vp, vp, vp, i32, vp, i32, vp, sz, vp]
        L.rwkvq_gemv_static.argtypes = [C.POINTER(Desc), vp, C.POINTER(Desc), vp, vp, vp, i32, vp, i32, vp]
        L.rwkvq_gemv_static_max_scratch_bytes.argtypes = []
        L.rwkvq_gemv_static_max_scratch_bytes.restype = sz
        L.rwkvq_dequant.argtypes = [C.POINTER(Desc), vp, vp, i32, vp]
        L.rwkvq_device_status.argtypes = [vp]
    if hasattr(L, "rwkvq_proxy_select"):
        L.rwkvq_proxy_workspace_bytes.argtypes = [i32]
        L.rwkvq_proxy_workspace_bytes.restype = sz
        L.rwkvq_proxy_select.argtypes = [C.POINTER(vp), C.POINTER(i32), C.POINTER(i32), i32, i32, dbl, dbl,
                                         C.POINTER(dbl), C.POINTER(dbl), C.POINTER(i32), vp, sz, vp]
    if hasattr(L, "rwkvq_proxy_family"):
        L.rwkvq_proxy_family.argtypes = [C.POINTER(vp), C.POINTER(i32), C.POINTER(i32), i32, C.POINTER(dbl), vp, sz, vp]
        L.rwkvq_tau_for_fraction.argtypes = [C.POINTER(dbl), i32, dbl, C.POINTER(dbl)]
        L.rwkvq_tau_largest_gap.argtypes = [C.POINTER(dbl), i32, C.POINTER(dbl)]
    if hasattr(L, "rwkvq_proxy_segments"):
        L.rwkvq_proxy_select_bf16.argtypes = L.rwkvq_proxy_select.argtypes
        L.rwkvq_proxy_f32_workspace_bytes.argtypes = [i32, i32]
        L.rwkvq_proxy_f32_workspace_bytes.restype = sz
        L.rwkvq_proxy_select_f32.argtypes = [vp, i32, i32, i32, dbl, dbl, C.POINTER(dbl), C.POINTER(dbl), C.POINTER(i32), vp, sz, vp]
        L.rwkvq_proxy_segments_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.rwkvq_proxy_segments_workspace_bytes.restype = sz
        L.rwkvq_proxy_segments.argtypes = [vp, i32, i32, i32, i32, i32, i32, dbl, dbl, C.POINTER(dbl), C.POINTER(dbl),
                                           C.POINTER(i32), vp, sz, vp]
    if hasattr(L, "rwkvq_quant_error"):
        L.rwkvq_quant_error_workspace_bytes.argtypes = [C.POINTER(Desc)]
        L.rwkvq_quant_error_workspace_bytes.restype = sz
        L.rwkvq_quant_error.argtypes = [vp, C.POINTER(Desc), vp, C.POINTER(dbl), vp, sz, vp]
    if hasattr(L, "rwkvq_step_plan"):
        L.rwkvq_step_plan_bytes.argtypes = [C.POINTER(GemvOp), i32, i32]
        L.rwkvq_step_plan_bytes.restype = sz
        L.rwkvq_step_plan.argtypes = [C.POINTER(GemvOp), i32, i32, vp, sz, vp]
        L.rwkvq_step_run.argtypes = [vp, sz, vp]
        L.rwkvq_step_run_host.argtypes = [vp, sz, vp, vp, sz, vp, vp, sz, vp]
        L.rwkvq_step_plan_release.argtypes = [vp]
        L.rwkvq_step_set_wait.argtypes = [vp, C.c_uint32, C.c_uint32]
        L.rwkvq_step_plan_cover.argtypes = [C.POINTER(GemvOp), i32, i32, i32, C.POINTER(C.c_uint32), sz, C.POINTER(C.c_uint32)]
    if hasattr(L, "rwkvq_gemm_prefill"):
        L.rwkvq_prefill_workspace_bytes.argtypes = [C.POINTER(Desc), i32, i32]
        L.rwkvq_prefill_workspace_bytes.restype = sz
        L.rwkvq_gemm_prefill.argtypes = [C.POINTER(Desc), vp, C.POINTER(Desc), vp, vp, vp, i32, vp, i32, vp, sz, vp]
        L.rwkvq_gemm_prefill_grouped.argtypes = [C.POINTER(PrefillOp), i32, i32, i32, vp]
    if hasattr(L, "rwkvq_quantize_dev"):
        L.rwkvq_desc_for.argtypes = [C.POINTER(QuantCfg), i32, i32, C.POINTER(Desc)]
        L.rwkvq_quantize_workspace_bytes.argtypes = []
        L.rwkvq_quantize_workspace_bytes.restype = sz
        L.rwkvq_quantize_dev.argtypes = [vp, i32, i32, C.POINTER(QuantCfg), vp, vp, sz, C.POINTER(Desc), vp, sz, vp]
        L.rwkvq_calib_representative.argtypes = [vp, i32, i32, dbl, vp, vp, vp]
        L.rwkvq_quantize_dev_async.argtypes = L.rwkvq_quantize_dev.argtypes
        L.rwkvq_quantize_check.argtypes = [vp, vp]
    _lib = L
    return L


def _check(status: int, where: str):
    if status != 0:
        raise RwkvqError(status, where)


def _np_ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dev_ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Blob:
    """Host-owned packed matrix (rwkvq_blob)."""

    def __init__(self, handle):
        self._h = C.c_void_p(handle)
        self.desc = Desc()
        _check(lib().rwkvq_blob_desc(self._h, C.byref(self.desc)), "rwkvq_blob_desc")

    def __del__(self):
        try:
            if self._h:
                lib().rwkvq_blob_free(self._h)
                self._h = None
        except Exception:
            pass

    @property
    def nbytes(self) -> int:
        return int(lib().rwkvq_blob_nbytes(self._h))

    def image(self) -> np.ndarray:
        """rwkvq_blob_image: the device image as a host uint8 array."""
        out = np.empty(self.nbytes, dtype=np.uint8)
        _check(lib().rwkvq_blob_image(self._h, _np_ptr(out), out.nbytes), "rwkvq_blob_image")
        return out

    def export_codes(self) -> dict:
        """rwkvq_blob_export_codes: logical codes as numpy arrays."""
        return _alloc_codes(self.desc, lambda c: lib().rwkvq_blob_export_codes(self._h, C.byref(c)),
                            "rwkvq_blob_export_codes")

    def to_device(self, device="cuda"):
        """Copy the image into a torch uint8 tensor on `device` (256-byte aligned by torch)."""
        import torch
        return torch.from_numpy(self.image()).to(device)


def _alloc_codes(d: Desc, call, where):
    out = {}
    c = Codes()
    if d.method == RWKVQ_SQ:
        ng = d.oc * (d.ic // d.group)
        out["q"] = np.empty((d.oc, d.ic), np.uint8)
        out["scale"] = np.empty((d.oc, d.ic // d.group), np.float16)
        out["zero"] = np.empty((d.oc, d.ic // d.group), np.float16)
        c.q, c.scale, c.zero = _np_ptr(out["q"]), _np_ptr(out["scale"]), _np_ptr(out["zero"])
        assert ng == out["scale"].size
    elif d.oc == 1:
        out["q"] = np.empty((d.ic // 2,), np.uint8)
        out["codebook"] = np.empty((d.entries, 2), np.float16)
        c.q, c.codebook = _np_ptr(out["q"]), _np_ptr(out["codebook"])
    else:
        out["q"] = np.empty((d.oc, d.ic // 2), np.uint8)
        out["codebook"] = np.empty((d.oc // d.tile, d.ic // d.tile, d.entries, 2), np.float16)
        c.q, c.codebook = _np_ptr(out["q"]), _np_ptr(out["codebook"])
    _check(call(c), where)
    return out


def rwkvq_pack(w16: np.ndarray | None, oc: int, ic: int, method: int, bits: int, *, group: int = 128,
               vec_dim: int = 2, tile: int = 256, kmeans_iters: int = 10, seed: int = 0,
               codes: dict | None = None) -> Blob:
    """rwkvq_pack.  `w16`: float16 [oc, ic] (or None with `codes`).  `codes`: logical codes as
    numpy arrays {q, scale, zero} (SQ) or {q, codebook} (VQ) to pack as given."""
    cfg = QuantCfg(method=method, bits=bits, group=group, vec_dim=vec_dim, tile=tile,
                   kmeans_iters=kmeans_iters, seed=seed, codes_in=None)
    keep = []
    if codes is not None:
        c = Codes()
        q = np.ascontiguousarray(codes["q"], dtype=np.uint8)
        keep.append(q)
        c.q = _np_ptr(q)
        if method == RWKVQ_SQ:
            s = np.ascontiguousarray(codes["scale"], dtype=np.float16)
            z = np.ascontiguousarray(codes["zero"], dtype=np.float16)
            keep += [s, z]
            c.scale, c.zero = _np_ptr(s), _np_ptr(z)
        else:
            cb = np.ascontiguousarray(codes["codebook"], dtype=np.float16)
            keep.append(cb)
            c.codebook = _np_ptr(cb)
        keep.append(c)
        cfg.codes_in = C.pointer(c)
    w = None
    if w16 is not None:
        w = np.ascontiguousarray(w16, dtype=np.float16)
        assert w.shape == (oc, ic) or w.size == oc * ic
    handle = C.c_void_p()
    _check(lib().rwkvq_pack(_np_ptr(w), oc, ic, C.byref(cfg), C.byref(handle)), "rwkvq_pack")
    return Blob(handle.value)


def rwkvq_image_unpack(image: np.ndarray):
    """rwkvq_image_unpack: (Desc, logical codes) from a host copy of a device image."""
    img = np.ascontiguousarray(image, dtype=np.uint8)
    d = Desc()
    _check(lib().rwkvq_image_unpack(_np_ptr(img), img.nbytes, C.byref(d), None), "rwkvq_image_unpack")
    codes = _alloc_codes(d, lambda c: lib().rwkvq_image_unpack(_np_ptr(img), img.nbytes, None, C.byref(c)),
                         "rwkvq_image_unpack")
    return d, codes


def rwkvq_gemv_workspace_bytes(desc: Desc, B: int) -> int:
    return int(lib().rwkvq_gemv_workspace_bytes(C.byref(desc), B))


def rwkvq_gemv(desc: Desc, W_image, mu_desc, mu_image, x, xprev, B: int, y, workspace, stream=None):
    """rwkvq_gemv on torch tensors: W_image/mu_image uint8, x/xprev float16 [B, ic], y float32 or
    float16 [B, oc], workspace uint8 (zero-filled before first use)."""
    import torch
    y_dtype = RWKVQ_F32 if y.dtype == torch.float32 else RWKVQ_F16
    _check(lib().rwkvq_gemv(C.byref(desc), _dev_ptr(W_image), None if mu_desc is None else C.byref(mu_desc),
                            _dev_ptr(mu_image), _dev_ptr(x), _dev_ptr(xprev), B, _dev_ptr(y), y_dtype,
                            _dev_ptr(workspace), workspace.numel() * workspace.element_size(),
                            _stream_ptr(stream)), "rwkvq_gemv")


def rwkvq_gemv_static_max_scratch_bytes() -> int:
    return int(lib().rwkvq_gemv_static_max_scratch_bytes())


def rwkvq_gemv_static(desc: Desc, W_image, mu_desc, mu_image, x, xprev, B: int, y, stream=None):
    """rwkvq_gemv_static: same product as rwkvq_gemv, scratch inside the library (no workspace)."""
    import torch
    y_dtype = RWKVQ_F32 if y.dtype == torch.float32 else RWKVQ_F16
    _check(lib().rwkvq_gemv_static(C.byref(desc), _dev_ptr(W_image), None if mu_desc is None else C.byref(mu_desc),
                                   _dev_ptr(mu_image), _dev_ptr(x), _dev_ptr(xprev), B, _dev_ptr(y), y_dtype,
                                   _stream_ptr(stream)), "rwkvq_gemv_static")


def rwkvq_dequant(desc: Desc, W_image, out, stream=None):
    """rwkvq_dequant into `out` (torch float32 or bfloat16, [oc, ic] or [ic])."""
    import torch
    dt = RWKVQ_F32 if out.dtype == torch.float32 else RWKVQ_BF16
    _check(lib().rwkvq_dequant(C.byref(desc), _dev_ptr(W_image), _dev_ptr(out), dt, _stream_ptr(stream)),
           "rwkvq_dequant")


def rwkvq_device_status(stream=None) -> int:
    return int(lib().rwkvq_device_status(_stream_ptr(stream)))


def rwkvq_proxy_workspace_bytes(n_mats: int) -> int:
    return int(lib().rwkvq_proxy_workspace_bytes(n_mats))


def rwkvq_proxy_select(mats, K: int, tau_c: float, tau_f: float, workspace, stream=None):
    """rwkvq_proxy_select on a list of torch float16 [oc, ic] device tensors.
    Returns (P_c, P_f, phi) numpy arrays."""
    n = len(mats)
    ptrs = (C.c_void_p * n)(*[m.data_ptr() for m in mats])
    ocs = (C.c_int * n)(*[m.shape[0] for m in mats])
    ics = (C.c_int * n)(*[m.shape[1] for m in mats])
    pc = np.empty(n, np.float64)
    pf = np.empty(n, np.float64)
    phi = np.empty(n, np.int32)
    _check(lib().rwkvq_proxy_select(ptrs, ocs, ics, n, K, tau_c, tau_f,
                                    pc.ctypes.data_as(C.POINTER(C.c_double)),
                                    pf.ctypes.data_as(C.POINTER(C.c_double)),
                                    phi.ctypes.data_as(C.POINTER(C.c_int)),
                                    _dev_ptr(workspace), workspace.numel() * workspace.element_size(),
                                    _stream_ptr(stream)), "rwkvq_proxy_select")
    return pc, pf, phi


def _torch_dtype_code(t):
    import torch
    return {torch.float32: RWKVQ_F32, torch.float16: RWKVQ_F16, torch.bfloat16: RWKVQ_BF16}[t.dtype]


def rwkvq_proxy_select_typed(w, K: int, tau_c: float, tau_f: float, stream=None):
    """P_c, P_f and phi of ONE matrix (CUDA tensor [oc, ic], float16, bfloat16 or float32) as floats / int:
    rwkvq_proxy_select, rwkvq_proxy_select_bf16 or rwkvq_proxy_select_f32 by the tensor's type."""
    import torch
    oc, ic = int(w.shape[0]), int(w.shape[1])
    pc, pf, phi = C.c_double(), C.c_double(), C.c_int()
    if w.dtype == torch.float32:
        ws = torch.empty(int(lib().rwkvq_proxy_f32_workspace_bytes(oc, ic)), dtype=torch.uint8, device=w.device)
        _check(lib().rwkvq_proxy_select_f32(_dev_ptr(w), oc, ic, K, tau_c, tau_f, C.byref(pc), C.byref(pf), C.byref(phi),
                                            _dev_ptr(ws), ws.numel(), _stream_ptr(stream)), "rwkvq_proxy_select_f32")
    else:
        ws = torch.empty(rwkvq_proxy_workspace_bytes(1), dtype=torch.uint8, device=w.device)
        fn = lib().rwkvq_proxy_select if w.dtype == torch.float16 else lib().rwkvq_proxy_select_bf16
        ptrs, ocs, ics = (C.c_void_p * 1)(w.data_ptr()), (C.c_int * 1)(oc), (C.c_int * 1)(ic)
        _check(fn(ptrs, ocs, ics, 1, K, tau_c, tau_f, C.byref(pc), C.byref(pf), C.byref(phi), _dev_ptr(ws), ws.numel(),
                  _stream_ptr(stream)), "rwkvq_proxy_select (typed)")
    return float(pc.value), float(pf.value), int(phi.value)


def rwkvq_proxy_segments(w, seg_rows: int, seg_cols: int, K: int, tau_c: float, tau_f: float, stream=None):
    """rwkvq_proxy_segments on a CUDA tensor [oc, ic] (float16, bfloat16 or float32).  Returns (P_c, P_f, phi)
    numpy arrays of shape [ceil(oc / seg_rows), ceil(ic / seg_cols)]."""
    import torch
    oc, ic = int(w.shape[0]), int(w.shape[1])
    sr, sc = min(seg_rows, oc), min(seg_cols, ic)
    gy, gx = (oc + sr - 1) // sr, (ic + sc - 1) // sc
    pc, pf, phi = np.empty(gy * gx, np.float64), np.empty(gy * gx, np.float64), np.empty(gy * gx, np.int32)
    ws = torch.empty(max(256, int(lib().rwkvq_proxy_segments_workspace_bytes(oc, ic, sr, sc))), dtype=torch.uint8, device=w.device)
    _check(lib().rwkvq_proxy_segments(_dev_ptr(w), _torch_dtype_code(w), oc, ic, seg_rows, seg_cols, K, tau_c, tau_f,
                                      pc.ctypes.data_as(C.POINTER(C.c_double)), pf.ctypes.data_as(C.POINTER(C.c_double)),
                                      phi.ctypes.data_as(C.POINTER(C.c_int)), _dev_ptr(ws), ws.numel(), _stream_ptr(stream)),
           "rwkvq_proxy_segments")
    return pc.reshape(gy, gx), pf.reshape(gy, gx), phi.reshape(gy, gx)


def rwkvq_proxy_family(mats, workspace, stream=None):
    """rwkvq_proxy_family on a list of torch float16 [oc, ic] device tensors.  Returns a dict of numpy
    arrays: variance, cv, range, mad, ie."""
    n = len(mats)
    ptrs = (C.c_void_p * n)(*[m.data_ptr() for m in mats])
    ocs = (C.c_int * n)(*[m.shape[0] for m in mats])
    ics = (C.c_int * n)(*[m.shape[1] for m in mats])
    stats = np.empty((n, 5), np.float64)
    _check(lib().rwkvq_proxy_family(ptrs, ocs, ics, n, stats.ctypes.data_as(C.POINTER(C.c_double)),
                                    _dev_ptr(workspace), workspace.numel() * workspace.element_size(),
                                    _stream_ptr(stream)), "rwkvq_proxy_family")
    return {k: stats[:, i].copy() for i, k in enumerate(("variance", "cv", "range", "mad", "ie"))}


def rwkvq_tau_for_fraction(values, sq_fraction: float) -> float:
    v = np.ascontiguousarray(values, dtype=np.float64)
    tau = C.c_double()
    _check(lib().rwkvq_tau_for_fraction(v.ctypes.data_as(C.POINTER(C.c_double)), v.size, float(sq_fraction),
                                        C.byref(tau)), "rwkvq_tau_for_fraction")
    return float(tau.value)


def rwkvq_tau_largest_gap(values) -> float:
    v = np.ascontiguousarray(values, dtype=np.float64)
    tau = C.c_double()
    _check(lib().rwkvq_tau_largest_gap(v.ctypes.data_as(C.POINTER(C.c_double)), v.size, C.byref(tau)),
           "rwkvq_tau_largest_gap")
    return float(tau.value)


def rwkvq_quant_error(w, desc: Desc, W_image, stream=None) -> float:
    """rwkvq_quant_error: sum of squared differences between the fp16 CUDA tensor `w` and the decoded image."""
    import torch
    ws = torch.empty(int(lib().rwkvq_quant_error_workspace_bytes(C.byref(desc))), dtype=torch.uint8, device=w.device)
    sse = C.c_double()
    _check(lib().rwkvq_quant_error(_dev_ptr(w), C.byref(desc), _dev_ptr(W_image), C.byref(sse), _dev_ptr(ws),
                                   ws.numel(), _stream_ptr(stream)), "rwkvq_quant_error")
    return float(sse.value)


def make_ops(entries):
    """Array of GemvOp from dicts {desc, W, mu_desc, mu, x, xprev, y, stage[, in]} (torch tensors; "in" is a
    dict describing an rwkvq_input_xform)."""
    import torch
    arr = (GemvOp * len(entries))()
    for i, e in enumerate(entries):
        o = arr[i]
        o.W_desc = e["desc"]
        o.W_image_dev = e["W"].data_ptr()
        if e.get("mu") is not None:
            o.mu_desc = e["mu_desc"]
            o.mu_image_dev = e["mu"].data_ptr()
            o.xprev_fp16_dev = e["xprev"].data_ptr()
        else:
            o.mu_image_dev = None
            o.xprev_fp16_dev = None
        o.x_fp16_dev = None if e.get("x") is None else e["x"].data_ptr()
        xf = e.get("in")
        if xf:      # {"kind": RWKVQ_IN_*, "src": .., "k": .., "v": .., "state_a": .., ..., "gate": .., "xprev_out": ..}
            o.in_.kind = int(xf.get("kind", RWKVQ_IN_BUFFER))
            o.in_.flags = RWKVQ_INF_RMSNORM if xf.get("rmsnorm") else 0
            for field, key in (("src_f32", "src"), ("k_f32", "k"), ("v_f32", "v"), ("state_a", "state_a"),
                               ("state_b", "state_b"), ("state_p", "state_p"), ("u_f32", "u"), ("w_f32", "w"),
                               ("gate_f32", "gate"), ("xprev_out_fp16", "xprev_out"), ("scale_f32", "scale")):
                t = xf.get(key)
                setattr(o.in_, field, None if t is None else t.data_ptr())
        o.y_dev = e["y"].data_ptr()
        o.stage = e["stage"]
        o.y_dtype = RWKVQ_F32 if e["y"].dtype == torch.float32 else RWKVQ_F16
    return arr


def rwkvq_step_plan_bytes(ops, B: int) -> int:
    return int(lib().rwkvq_step_plan_bytes(ops, len(ops), B))


def rwkvq_step_plan(ops, B: int, plan, stream=None):
    _check(lib().rwkvq_step_plan(ops, len(ops), B, _dev_ptr(plan), plan.numel(), _stream_ptr(stream)),
           "rwkvq_step_plan")


def rwkvq_step_run(plan, stream=None):
    _check(lib().rwkvq_step_run(_dev_ptr(plan), plan.numel(), _stream_ptr(stream)), "rwkvq_step_run")


def rwkvq_step_plan_release(plan):
    _check(lib().rwkvq_step_plan_release(_dev_ptr(plan)), "rwkvq_step_plan_release")


def rwkvq_step_set_wait(plan, poll_limit: int = 0, wait_skew: int = 0):
    _check(lib().rwkvq_step_set_wait(_dev_ptr(plan), poll_limit, wait_skew), "rwkvq_step_set_wait")


def rwkvq_step_plan_cover(ops, B: int, n_ctas: int):
    """Host-only walk of the schedule: (counts per (product, 16-row slice, column tile) as one flat
    numpy array in product order, records per CTA)."""
    import numpy as np
    n = sum((o.W_desc.oc // 16) * (o.W_desc.ic_pad // 256) for o in ops)
    counts = np.zeros(max(n, 1), dtype=np.uint32)
    per_cta = np.zeros(n_ctas, dtype=np.uint32)
    _check(lib().rwkvq_step_plan_cover(ops, len(ops), B, n_ctas, counts.ctypes.data_as(C.POINTER(C.c_uint32)), counts.size,
                                       per_cta.ctypes.data_as(C.POINTER(C.c_uint32))), "rwkvq_step_plan_cover")
    return counts[:n], per_cta


def rwkvq_step_run_host(plan, act_host, act_dev, y_dev, y_host, stream=None):
    """rwkvq_step_run_host: act_host / y_host are (pinned) host uint8 tensors, act_dev / y_dev the
    device buffers the plan's activations and outputs lie in."""
    _check(lib().rwkvq_step_run_host(_dev_ptr(plan), plan.numel(), C.c_void_p(act_host.data_ptr()),
                                     _dev_ptr(act_dev), act_host.numel(), _dev_ptr(y_dev),
                                     C.c_void_p(y_host.data_ptr()), y_host.numel(), _stream_ptr(stream)),
           "rwkvq_step_run_host")


def rwkvq_prefill_workspace_bytes(desc: Desc, M: int, has_mu: bool) -> int:
    return int(lib().rwkvq_prefill_workspace_bytes(C.byref(desc), M, 1 if has_mu else 0))


def rwkvq_gemm_prefill(desc: Desc, W_image, mu_desc, mu_image, X, xprev0, M: int, Y, workspace, stream=None):
    """rwkvq_gemm_prefill: X bfloat16 [M, ic], Y float32 or bfloat16 [M, oc]."""
    import torch
    dt = RWKVQ_F32 if Y.dtype == torch.float32 else RWKVQ_BF16
    _check(lib().rwkvq_gemm_prefill(C.byref(desc), _dev_ptr(W_image), None if mu_desc is None else C.byref(mu_desc),
                                    _dev_ptr(mu_image), _dev_ptr(X), _dev_ptr(xprev0), M, _dev_ptr(Y), dt,
                                    _dev_ptr(workspace),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream_ptr(stream)), "rwkvq_gemm_prefill")


def make_prefill_ops(entries):
    """entries: dicts with desc, W, mu_desc, mu, X, xprev0, Y, workspace (CUDA tensors or None).  Returns
    (array of PrefillOp, objects to keep alive while the array is in use)."""
    arr = (PrefillOp * len(entries))()
    keep = []
    for o, e in zip(arr, entries):
        o.W_desc = C.pointer(e["desc"])
        o.W_image_dev = _dev_ptr(e["W"])
        md = e.get("mu_desc")
        if md is not None:
            o.mu_desc = C.pointer(md)
        o.mu_image_dev = _dev_ptr(e.get("mu"))
        o.X_bf16_dev = _dev_ptr(e["X"])
        o.xprev0_bf16_dev = _dev_ptr(e.get("xprev0"))
        o.Y_dev = _dev_ptr(e["Y"])
        ws = e.get("workspace")
        o.workspace_dev = _dev_ptr(ws)
        o.workspace_bytes = 0 if ws is None else ws.numel() * ws.element_size()
        keep.append(e)
    return arr, keep


def rwkvq_gemm_prefill_grouped(ops, M: int, y_dtype: int = RWKVQ_F32, stream=None):
    """rwkvq_gemm_prefill_grouped on an array from make_prefill_ops (or a list of entry dicts)."""
    if isinstance(ops, (list, tuple)):
        ops, _keep = make_prefill_ops(ops)
    _check(lib().rwkvq_gemm_prefill_grouped(ops, len(ops), M, y_dtype, _stream_ptr(stream)), "rwkvq_gemm_prefill_grouped")


def rwkvq_desc_for(oc: int, ic: int, method: int, bits: int, *, group: int = 128, vec_dim: int = 2,
                   tile: int = 256) -> Desc:
    cfg = QuantCfg(method=method, bits=bits, group=group, vec_dim=vec_dim, tile=tile, kmeans_iters=0, seed=0,
                   codes_in=None)
    d = Desc()
    _check(lib().rwkvq_desc_for(C.byref(cfg), oc, ic, C.byref(d)), "rwkvq_desc_for")
    return d


def rwkvq_quantize_workspace_bytes() -> int:
    return int(lib().rwkvq_quantize_workspace_bytes())


def rwkvq_quantize_dev(w, oc: int, ic: int, method: int, bits: int, image, workspace, *, elem_weight=None,
                       group: int = 128, vec_dim: int = 2, tile: int = 256, kmeans_iters: int = 10, seed: int = 0,
                       stream=None) -> Desc:
    """rwkvq_quantize_dev.  `w`: float16 CUDA tensor [oc, ic]; `image`: uint8 CUDA tensor that receives
    the packed image; `elem_weight`: float32 CUDA tensor [ic] (vectors only) or None."""
    cfg = QuantCfg(method=method, bits=bits, group=group, vec_dim=vec_dim, tile=tile, kmeans_iters=kmeans_iters,
                   seed=seed, codes_in=None)
    d = Desc()
    _check(lib().rwkvq_quantize_dev(_dev_ptr(w), oc, ic, C.byref(cfg), _dev_ptr(elem_weight), _dev_ptr(image),
                                    image.numel() * image.element_size(), C.byref(d), _dev_ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
           "rwkvq_quantize_dev")
    return d


def rwkvq_quantize_dev_async(w, oc: int, ic: int, method: int, bits: int, image, workspace, *, elem_weight=None,
                             group: int = 128, vec_dim: int = 2, tile: int = 256, kmeans_iters: int = 10,
                             seed: int = 0, stream=None) -> Desc:
    """rwkvq_quantize_dev_async: enqueue only; `workspace` must have been zero-filled once."""
    cfg = QuantCfg(method=method, bits=bits, group=group, vec_dim=vec_dim, tile=tile, kmeans_iters=kmeans_iters,
                   seed=seed, codes_in=None)
    d = Desc()
    _check(lib().rwkvq_quantize_dev_async(_dev_ptr(w), oc, ic, C.byref(cfg), _dev_ptr(elem_weight), _dev_ptr(image),
                                          image.numel() * image.element_size(), C.byref(d), _dev_ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
           "rwkvq_quantize_dev_async")
    return d


def rwkvq_quantize_check(workspace, stream=None) -> int:
    """rwkvq_quantize_check: status code (0 = OK, 4 = a NaN/Inf weight was seen); synchronizes."""
    return int(lib().rwkvq_quantize_check(_dev_ptr(workspace), _stream_ptr(stream)))


def rwkvq_calib_representative(samples, pct: float, rep=None, rep_sq=None, stream=None):
    """rwkvq_calib_representative.  `samples`: float32 CUDA tensor [n_samples, n]."""
    S, n = samples.shape
    _check(lib().rwkvq_calib_representative(_dev_ptr(samples), S, n, float(pct), _dev_ptr(rep), _dev_ptr(rep_sq),
                                            _stream_ptr(stream)), "rwkvq_calib_representative")
