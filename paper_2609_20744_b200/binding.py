"""Thin ctypes binding over the C ABI declared in include/vdn_vda.h.

Argument marshalling only: every step of the layer runs inside the CUDA library.  torch is used
for device memory and streams.  There is no CPU fallback: if the shared library is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("VDN_VDA_LIB") or os.path.join(_HERE, "libvdn_vda.so")   # VDN_VDA_LIB: another build of the library

VDN_OK = 0
STATUS_NAMES = {0: "VDN_OK", 1: "VDN_ERR_INVALID_ARG", 2: "VDN_ERR_UNSUPPORTED", 3: "VDN_ERR_WORKSPACE",
                4: "VDN_ERR_CUDA", 5: "VDN_ERR_ARCH", 6: "VDN_ERR_TIMEOUT", 7: "VDN_ERR_INTERNAL"}
VDN_ERR_TIMEOUT, VDN_ERR_INTERNAL = 6, 7
VDN_F32, VDN_BF16 = 0, 1
VDN_FLAG_FORCE_SIMT = 1
VDN_FLAG_ADDITIVE_RULE = 4
VDN_FLAG_SCAN_CHUNKWISE = 8
VDN_FLAG_SCAN_FRAMEWISE = 16
VDN_FLAG_EXACT_STATS = 32
VDN_FLAG_FP32_RESOLVE = 64
VIEW_STATS, VIEW_INV, VIEW_FWD, VIEW_READ, VIEW_INV_SPLIT, VIEW_READ_FWD, VIEW_READ_BWD, VIEW_COMP_M, VIEW_COMP_J = range(9)

EXPORTS = (
    "vdn_vda_create", "vdn_vda_workspace_bytes", "vdn_vda_set_workspace", "vdn_vda_forward", "vdn_vda_forward_ex",
    "vdn_vda_forward_opt", "vdn_vda_workspace_bytes_opt", "vdn_vda_prepare",
    "vdn_vda_staging_bytes", "vdn_vda_staging_bytes_opt", "vdn_vda_set_staging", "vdn_vda_forward_host",
    "vdn_vda_forward_host_opt", "vdn_vda_workspace_view",
    "vdn_vda_last_launch_count", "vdn_vda_profile", "vdn_vda_kernel_times", "vdn_vda_scan_static", "vdn_vda_status",
    "vdn_vda_clear_status", "vdn_vda_set_wait_limit_us", "vdn_vda_selftest_wait_expiry", "vdn_vda_selftest_marker",
    "vdn_vda_last_error", "vdn_vda_destroy",
)


class VdnConfig(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("io_dtype", ctypes.c_int32), ("d", ctypes.c_int32),
                ("rms_eps", ctypes.c_float), ("flags", ctypes.c_uint32), ("device", ctypes.c_int32)]


class VdnOptions(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("chunk", ctypes.c_int32), ("radius", ctypes.c_int32),
                ("anchors", ctypes.c_int32), ("alpha", ctypes.c_void_p), ("s0", ctypes.c_void_p),
                ("gate_elem", ctypes.c_void_p), ("norm_weight", ctypes.c_void_p), ("q_l2_eps", ctypes.c_float),
                ("reserved", ctypes.c_uint32)]


class VdnPrepParams(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("Y", ctypes.c_int32), ("X", ctypes.c_int32),
                ("anchors", ctypes.c_int32), ("l2_eps", ctypes.c_float), ("wk_spatial", ctypes.c_void_p),
                ("wk_temporal", ctypes.c_void_p), ("wv_spatial", ctypes.c_void_p), ("wv_temporal", ctypes.c_void_p)]


class VdnError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """dlopen the CUDA library and declare its signatures.  Raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2609_20744_b200.build` (there is no CPU fallback)")
    lib = ctypes.CDLL(p)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    shape = [ci, ci, ci, ci, ci]
    lib.vdn_vda_create.argtypes = [ctypes.POINTER(VdnConfig), ctypes.POINTER(vp)]
    lib.vdn_vda_create.restype = ci
    lib.vdn_vda_workspace_bytes.argtypes = [vp, *shape]
    lib.vdn_vda_workspace_bytes.restype = sz
    lib.vdn_vda_set_workspace.argtypes = [vp, vp, sz]
    lib.vdn_vda_set_workspace.restype = ci
    lib.vdn_vda_staging_bytes.argtypes = [vp, *shape]
    lib.vdn_vda_staging_bytes.restype = sz
    lib.vdn_vda_set_staging.argtypes = [vp, vp, sz]
    lib.vdn_vda_set_staging.restype = ci
    fwd_args = [vp, vp, vp, vp, vp, vp, vp, *shape, vp]
    lib.vdn_vda_forward.argtypes = fwd_args
    lib.vdn_vda_forward.restype = ci
    lib.vdn_vda_forward_ex.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, *shape, vp]
    lib.vdn_vda_forward_ex.restype = ci
    lib.vdn_vda_forward_opt.argtypes = [vp, vp, vp, vp, vp, vp, vp, *shape, ctypes.POINTER(VdnOptions), vp]
    lib.vdn_vda_forward_opt.restype = ci
    lib.vdn_vda_workspace_bytes_opt.argtypes = [vp, *shape, ctypes.POINTER(VdnOptions)]
    lib.vdn_vda_workspace_bytes_opt.restype = sz
    lib.vdn_vda_prepare.argtypes = [vp, vp, vp, vp, vp, vp, vp, *shape, ctypes.POINTER(VdnPrepParams), vp]
    lib.vdn_vda_prepare.restype = ci
    lib.vdn_vda_forward_host.argtypes = fwd_args
    lib.vdn_vda_forward_host.restype = ci
    lib.vdn_vda_forward_host_opt.argtypes = [vp, vp, vp, vp, vp, vp, vp, *shape, ctypes.POINTER(VdnOptions), vp]
    lib.vdn_vda_forward_host_opt.restype = ci
    lib.vdn_vda_staging_bytes_opt.argtypes = [vp, *shape, ctypes.POINTER(VdnOptions)]
    lib.vdn_vda_staging_bytes_opt.restype = sz
    lib.vdn_vda_clear_status.argtypes = [vp]
    lib.vdn_vda_clear_status.restype = ci
    lib.vdn_vda_set_wait_limit_us.argtypes = [vp, ctypes.c_ulonglong]
    lib.vdn_vda_set_wait_limit_us.restype = ci
    lib.vdn_vda_selftest_wait_expiry.argtypes = [vp, ctypes.c_ulonglong, vp]
    lib.vdn_vda_selftest_wait_expiry.restype = ci
    lib.vdn_vda_selftest_marker.argtypes = [vp]
    lib.vdn_vda_selftest_marker.restype = ci
    lib.vdn_vda_workspace_view.argtypes = [vp, ci, *shape, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.vdn_vda_workspace_view.restype = ci
    lib.vdn_vda_last_launch_count.argtypes = [vp]
    lib.vdn_vda_last_launch_count.restype = ci
    lib.vdn_vda_profile.argtypes = [vp, ci]
    lib.vdn_vda_profile.restype = ci
    lib.vdn_vda_kernel_times.argtypes = [vp, ci, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float),
                                         ctypes.POINTER(ci)]
    lib.vdn_vda_kernel_times.restype = ci
    lib.vdn_vda_scan_static.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, ctypes.c_char_p, sz]
    lib.vdn_vda_scan_static.restype = ci
    lib.vdn_vda_status.argtypes = [vp]
    lib.vdn_vda_status.restype = ci
    lib.vdn_vda_last_error.argtypes = [vp]
    lib.vdn_vda_last_error.restype = ctypes.c_char_p
    lib.vdn_vda_destroy.argtypes = [vp]
    lib.vdn_vda_destroy.restype = ci
    if path is None:
        _lib = lib
    return lib


SCAN_STATIC_MAX_BYTES = 8 << 20


def scan_static(stats, inv, read, stream=None):
    """vdn_vda_scan_static: the fp32 frame scan + gather with its scratch inside the library image.

    For callers that may not allocate device memory.  stats [BH,T,2d,d], inv [BH,T,d,d] and the output
    read [BH,T,d,d] are contiguous float CUDA tensors owned by the caller; nothing is allocated here or
    in the library.  Raises VdnError (VDN_ERR_WORKSPACE) when BH*T*d*d*4 exceeds SCAN_STATIC_MAX_BYTES.
    Calls that may overlap on the GPU share the scratch and must be serialised by the caller.
    """
    import torch
    lib = load_library()
    BH, T, d2, d = stats.shape
    for x in (stats, inv, read):
        if not (x.is_cuda and x.is_contiguous() and x.dtype == torch.float32):
            raise ValueError("scan_static needs contiguous float32 CUDA tensors")
    if d2 != 2 * d or tuple(inv.shape) != (BH, T, d, d) or tuple(read.shape) != (BH, T, d, d):
        raise ValueError("scan_static: shapes must be stats [BH,T,2d,d], inv/read [BH,T,d,d]")
    dev = stats.device.index or 0
    s = stream if stream is not None else torch.cuda.current_stream(dev)
    err = ctypes.create_string_buffer(256)
    st = lib.vdn_vda_scan_static(ctypes.c_void_p(stats.data_ptr()), ctypes.c_void_p(inv.data_ptr()),
                                 ctypes.c_void_p(read.data_ptr()), BH, T, d, dev, ctypes.c_void_p(s.cuda_stream),
                                 err, len(err))
    if st != VDN_OK:
        raise VdnError(st, err.value.decode())
    return read


def _require(name, x, shape, dtype, on_cuda, device_index):
    """One tensor argument against what the C ABI will assume about it (the library sees only a pointer)."""
    if x is None:
        raise ValueError(f"{name} is missing")
    where = "CUDA" if on_cuda else "host"
    if bool(x.is_cuda) != on_cuda:
        raise ValueError(f"{name} must be a {where} tensor")
    if on_cuda and (x.device.index or 0) != device_index:
        raise ValueError(f"{name} is on cuda:{x.device.index}, the handle is bound to cuda:{device_index}")
    if not x.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if x.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {x.dtype}")
    if tuple(x.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(x.shape)}")


def validate_layer_args(io_dtype, d_handle, device_index, q, k, v, beta, gate, out=None, alpha=None, s0=None,
                        gate_elem=None, norm_weight=None, on_cuda=True):
    """Checks every tensor of a forward call before anything reaches the library: dtype, shape, device and
    contiguity.  The kernels and the TMA tensor maps index by the shape that is passed, so a tensor of another dtype
    or a shorter one would be read (and `out` written) past its end.  Raises ValueError; returns (B, T, F, H, d).

    io_dtype is the torch dtype of the handle's q, k, v, out; on_cuda = False checks host tensors instead
    (the host-buffer entry point)."""
    import torch
    if q is None or q.dim() != 5:
        raise ValueError("q must have shape [B, T, F, H, d]")
    B, T, F, H, d = (int(n) for n in q.shape)
    del d_handle                      # a head dimension other than the handle's is the library's to refuse
    f32 = torch.float32
    _require("q", q, (B, T, F, H, d), io_dtype, on_cuda, device_index)
    _require("k", k, (B, T, F, H, d), io_dtype, on_cuda, device_index)
    _require("v", v, (B, T, F, H, d), io_dtype, on_cuda, device_index)
    _require("beta", beta, (B, T, F, H), f32, on_cuda, device_index)
    if gate is None and gate_elem is None:
        raise ValueError("gate may only be left out when gate_elem is given")
    if gate is not None:
        _require("gate", gate, (H,), f32, on_cuda, device_index)
    if out is not None:
        _require("out", out, (B, T, F, H, d), io_dtype, on_cuda, device_index)
    if alpha is not None:
        _require("alpha", alpha, (B, T, H, d), f32, on_cuda, device_index)
    if s0 is not None:
        _require("s0", s0, (B, H, d, d), f32, on_cuda, device_index)
    if gate_elem is not None:
        _require("gate_elem", gate_elem, (B, T, F, H, d), io_dtype, on_cuda, device_index)
    if norm_weight is not None:
        _require("norm_weight", norm_weight, (H, d), f32, on_cuda, device_index)
    return B, T, F, H, d


class Vda:
    """One handle of the library (vdn_vda_create .. vdn_vda_destroy) plus its torch-owned workspace."""

    def __init__(self, d: int, dtype: str = "bf16", rms_eps: float = 1e-6, flags: int = 0, device: int = 0):
        import torch
        self._torch = torch
        self.lib = load_library()
        self.d = d
        self.dtype = dtype
        self.torch_dtype = torch.float32 if dtype == "f32" else torch.bfloat16
        self.device = device
        cfg = VdnConfig(ctypes.sizeof(VdnConfig), VDN_F32 if dtype == "f32" else VDN_BF16, d, rms_eps, flags, device)
        self.h = ctypes.c_void_p()
        st = self.lib.vdn_vda_create(ctypes.byref(cfg), ctypes.byref(self.h))
        if st != VDN_OK:
            self.h = None
            raise VdnError(st, "vdn_vda_create failed")
        self._ws = None
        self._staging = None

    # -- helpers ------------------------------------------------------------------------------
    def _check(self, st: int):
        if st != VDN_OK:
            raise VdnError(st, self.lib.vdn_vda_last_error(self.h).decode())

    def _stream(self, stream):
        torch = self._torch
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        return ctypes.c_void_p(s.cuda_stream)

    def workspace_bytes(self, B, T, F, H, chunk=1) -> int:
        if chunk > 1:
            opt = VdnOptions(ctypes.sizeof(VdnOptions), chunk, 0, 0, None, None, None, None)
            return int(self.lib.vdn_vda_workspace_bytes_opt(self.h, B, T, F, H, self.d, ctypes.byref(opt)))
        return int(self.lib.vdn_vda_workspace_bytes(self.h, B, T, F, H, self.d))

    def ensure_workspace(self, B, T, F, H, chunk=1):
        torch = self._torch
        need = self.workspace_bytes(B, T, F, H, chunk)
        if need == 0:
            raise VdnError(1, "invalid shape")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}")
            self._check(self.lib.vdn_vda_set_workspace(self.h, ctypes.c_void_p(self._ws.data_ptr()), need))
        return self._ws

    def ensure_staging(self, B, T, F, H, opt=None):
        torch = self._torch
        if opt is None:
            need = int(self.lib.vdn_vda_staging_bytes(self.h, B, T, F, H, self.d))
        else:
            need = int(self.lib.vdn_vda_staging_bytes_opt(self.h, B, T, F, H, self.d, ctypes.byref(opt)))
        if need == 0:
            raise VdnError(1, "invalid shape")
        if self._staging is None or self._staging.numel() < need:
            self._staging = torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}")
            self._check(self.lib.vdn_vda_set_staging(self.h, ctypes.c_void_p(self._staging.data_ptr()), need))
        return self._staging

    # -- the two entry points -----------------------------------------------------------------
    def forward(self, q, k, v, beta, gate, out=None, stream=None, alpha=None, s0=None,
                chunk=1, radius=0, anchors=False, gate_elem=None, norm_weight=None, q_l2_eps=0.0):
        """vdn_vda_forward on device tensors q,k,v [B,T,F,H,d], beta [B,T,F,H], gate [H].

        With alpha [B,T,H,d] (decay gates) and/or s0 [B,H,d,d] (text state) the call goes to vdn_vda_forward_ex;
        with a chunk window (chunk, radius), boundary anchors, an element-wise gate gate_elem [B,T,F,H,d] (then
        `gate` may be None), a norm weight norm_weight [H,d] or q_l2_eps > 0 (q arrives without its L2
        normalisation; the read-out applies it) it goes to vdn_vda_forward_opt.
        """
        torch = self._torch
        B, T, F, H, d = validate_layer_args(self.torch_dtype, self.d, self.device, q, k, v, beta, gate, out, alpha, s0,
                                            gate_elem, norm_weight)
        if out is None:
            out = torch.empty_like(q)
        self.ensure_workspace(B, T, F, H, chunk)
        p = lambda x: ctypes.c_void_p(x.data_ptr()) if x is not None else None
        a = lambda x: x.data_ptr() if x is not None else None
        if (chunk, radius, bool(anchors)) != (1, 0, False) or gate_elem is not None or norm_weight is not None \
                or gate is None or q_l2_eps:
            opt = VdnOptions(ctypes.sizeof(VdnOptions), chunk, radius, 1 if anchors else 0, a(alpha), a(s0),
                             a(gate_elem), a(norm_weight), float(q_l2_eps), 0)
            st = self.lib.vdn_vda_forward_opt(self.h, p(q), p(k), p(v), p(beta), p(gate), p(out),
                                              B, T, F, H, d, ctypes.byref(opt), self._stream(stream))
        elif alpha is not None or s0 is not None:
            st = self.lib.vdn_vda_forward_ex(self.h, p(q), p(k), p(v), p(beta), p(gate), p(alpha), p(s0), p(out),
                                             B, T, F, H, d, self._stream(stream))
        else:
            st = self.lib.vdn_vda_forward(self.h, p(q), p(k), p(v), p(beta), p(gate), p(out),
                                          B, T, F, H, d, self._stream(stream))
        self._check(st)
        return out

    def prepare(self, q, k, v, filters, Y, X, anchors=False, l2_eps=1e-6, out=None, stream=None):
        """vdn_vda_prepare: projected q, k, v [B,T,F,H,d] -> prepared (q', k', v') (Sec. 2.3).

        filters = dict(wk_spatial [H*d,5,5], wk_temporal [H*d,5], wv_spatial, wv_temporal), float32 CUDA tensors.
        `out` = optional (q_out, k_out, v_out); q_out may be q itself.  q may be None: the queries are then left
        to the read-out (forward(..., q_l2_eps=l2_eps)) and the first element of the result is None.
        """
        torch = self._torch
        if k is None or k.dim() != 5:
            raise ValueError("k must have shape [B, T, F, H, d]")
        B, T, F, H, d = (int(n) for n in k.shape)
        names = ("wk_spatial", "wk_temporal", "wv_spatial", "wv_temporal")
        given = [n for n in names if filters.get(n) is not None]      # spatial filters may be left out (identity)
        for n, x in (("q", q), ("k", k), ("v", v)):
            if x is not None:
                _require(n, x, (B, T, F, H, d), self.torch_dtype, True, self.device)
        for n in given:
            want = (H * d, 5, 5) if n.endswith("spatial") else (H * d, 5)
            _require(n, filters[n], want, torch.float32, True, self.device)
        qo, ko, vo = out if out is not None else (torch.empty_like(q) if q is not None else None,
                                                  torch.empty_like(k), torch.empty_like(v))
        for n, x in (("q_out", qo), ("k_out", ko), ("v_out", vo)):
            if x is not None:
                _require(n, x, (B, T, F, H, d), self.torch_dtype, True, self.device)
        p = lambda x: ctypes.c_void_p(x.data_ptr()) if x is not None else None
        prm = VdnPrepParams(ctypes.sizeof(VdnPrepParams), Y, X, 1 if anchors else 0, l2_eps,
                            *(filters[n].data_ptr() if filters.get(n) is not None else None for n in names))
        self._check(self.lib.vdn_vda_prepare(self.h, p(q), p(k), p(v), p(qo), p(ko), p(vo), B, T, F, H, d,
                                             ctypes.byref(prm), self._stream(stream)))
        return qo, ko, vo

    def forward_host(self, q, k, v, beta, gate, out, stream=None, alpha=None, s0=None, chunk=1, radius=0,
                     anchors=False, gate_elem=None, norm_weight=None, q_l2_eps=0.0):
        """vdn_vda_forward_host(_opt) on HOST tensors (pinned recommended); `out` and every optional input are host
        tensors too.  The keyword arguments are those of forward()."""
        B, T, F, H, d = validate_layer_args(self.torch_dtype, self.d, self.device, q, k, v, beta, gate, out, alpha, s0,
                                            gate_elem, norm_weight, on_cuda=False)
        self.ensure_workspace(B, T, F, H, chunk)
        p = lambda x: ctypes.c_void_p(x.data_ptr()) if x is not None else None
        a = lambda x: x.data_ptr() if x is not None else None
        plain = (chunk, radius, bool(anchors)) == (1, 0, False) and gate is not None and not q_l2_eps and \
            all(x is None for x in (alpha, s0, gate_elem, norm_weight))
        opt = VdnOptions(ctypes.sizeof(VdnOptions), chunk, radius, 1 if anchors else 0, a(alpha), a(s0),
                         a(gate_elem), a(norm_weight), float(q_l2_eps), 0)
        self.ensure_staging(B, T, F, H, None if plain else opt)
        if plain:
            st = self.lib.vdn_vda_forward_host(self.h, p(q), p(k), p(v), p(beta), p(gate), p(out),
                                               B, T, F, H, d, self._stream(stream))
        else:
            st = self.lib.vdn_vda_forward_host_opt(self.h, p(q), p(k), p(v), p(beta), p(gate), p(out),
                                                   B, T, F, H, d, ctypes.byref(opt), self._stream(stream))
        self._check(st)
        return out

    # -- inspection ---------------------------------------------------------------------------
    def view(self, which: int, B, T, F, H):
        """A torch view of a workspace intermediate (valid after synchronising the stream)."""
        torch = self._torch
        off, size = ctypes.c_size_t(), ctypes.c_size_t()
        self._check(self.lib.vdn_vda_workspace_view(self.h, which, B, T, F, H, self.d,
                                                    ctypes.byref(off), ctypes.byref(size)))
        raw = self._ws[off.value: off.value + size.value]
        d = self.d
        if which == VIEW_STATS:
            return raw.view(torch.float32).view(B, H, T, 2 * d, d)
        if which == VIEW_INV_SPLIT:
            return raw.view(torch.bfloat16).view(B, H, T, 3, d, d)
        if which in (VIEW_READ_FWD, VIEW_READ_BWD):
            return raw.view(torch.bfloat16).view(B, H, T, d, d)
        if which == VIEW_COMP_M:
            return raw.view(torch.bfloat16).view(B * H, 2, -1, 3, d, d)
        if which == VIEW_COMP_J:
            return raw.view(torch.float32).view(B * H, 2, -1, d, d)
        return raw.view(torch.float32).view(B, H, T, d, d)

    def uses_tensor_cores(self) -> bool:
        """True when this handle runs the tcgen05 kernels (bf16 I/O, d = 128, plain-fp32 path not forced)."""
        off, size = ctypes.c_size_t(), ctypes.c_size_t()
        return self.lib.vdn_vda_workspace_view(self.h, VIEW_INV_SPLIT, 1, 1, 1, 1, self.d,
                                               ctypes.byref(off), ctypes.byref(size)) == VDN_OK

    def profile(self, enable: bool = True):
        """Start (and reset) or stop per-kernel CUDA-event timing of forward calls."""
        self._check(self.lib.vdn_vda_profile(self.h, 1 if enable else 0))

    def kernel_times(self):
        """[(kernel name, mean ms per launch, launches)] since profile(True); waits for the events."""
        n = 8
        names = (ctypes.c_char_p * n)()
        ms = (ctypes.c_float * n)()
        cnt = (ctypes.c_int * n)()
        got = self.lib.vdn_vda_kernel_times(self.h, n, names, ms, cnt)
        return [(names[i].decode(), float(ms[i]), int(cnt[i])) for i in range(got)]

    def launch_count(self) -> int:
        return int(self.lib.vdn_vda_last_launch_count(self.h))

    def status(self) -> int:
        return int(self.lib.vdn_vda_status(self.h))

    def clear_status(self) -> int:
        """Resets the sticky device-side status word; returns what it held."""
        return int(self.lib.vdn_vda_clear_status(self.h))

    def set_wait_limit_us(self, microseconds: int):
        """Longest single wait inside a kernel before its CTA gives up (default 2 s)."""
        self._check(self.lib.vdn_vda_set_wait_limit_us(self.h, int(microseconds)))

    def selftest_wait_expiry(self, limit_us: int = 1000, stream=None):
        """Enqueues the stand-alone kernel whose wait runs out (see vdn_vda_selftest_wait_expiry)."""
        self._check(self.lib.vdn_vda_selftest_wait_expiry(self.h, int(limit_us), self._stream(stream)))

    def selftest_marker(self) -> int:
        return int(self.lib.vdn_vda_selftest_marker(self.h))

    def close(self):
        if getattr(self, "h", None):
            self.lib.vdn_vda_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
