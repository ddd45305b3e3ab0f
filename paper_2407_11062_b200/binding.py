"""ctypes binding of libeqat_b200.so: same names as include/eqat.h.

Argument marshalling only.  Every function takes torch CUDA tensors (used as
device buffers), passes their data pointers and the current CUDA stream to the
C ABI and raises ``EqatError`` on a non-zero status.  Nothing is computed
here, and there is no fallback: if the library has not been built, importing
this module raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libeqat_b200.so")

EQAT_OK = 0
EQAT_ERR_NULL, EQAT_ERR_SHAPE, EQAT_ERR_ALIGN, EQAT_ERR_UNSUPPORTED = -1, -2, -3, -4
EQAT_ERR_WORKSPACE, EQAT_ERR_CUDA, EQAT_ERR_TIMEOUT = -5, -6, -7
EQAT_OP_FAKEQUANT_BWD, EQAT_OP_PACKED_BWD_DS = 1, 2
EQAT_ZP_U8, EQAT_ZP_FP16 = 0, 1


class EqatError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class eqat_desc(Structure):
    _fields_ = [("bits", c_int32), ("group", c_int32), ("out_features", c_int32), ("in_features", c_int32),
                ("tokens", c_int64), ("dz_mode", c_int32), ("zero_point_format", c_int32)]


class eqat_block_ap_linear(Structure):
    _fields_ = [("desc", eqat_desc), ("X", c_void_p), ("dY", c_void_p), ("W", c_void_p), ("s", c_void_p), ("z", c_void_p),
                ("Y", c_void_p), ("W_hat", c_void_p), ("dX", c_void_p), ("dW", c_void_p), ("ds", c_void_p),
                ("dz", c_void_p), ("workspace", c_void_p), ("workspace_bytes", c_size_t)]


class eqat_e2e_qp_linear(Structure):
    _fields_ = [("desc", eqat_desc), ("X", c_void_p), ("dY", c_void_p), ("Wq_packed", c_void_p), ("s16", c_void_p),
                ("z", c_void_p), ("Y", c_void_p), ("dX", c_void_p), ("ds", c_void_p), ("dz", c_void_p),
                ("workspace", c_void_p), ("workspace_bytes", c_size_t)]


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2407_11062_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(_LIB_PATH)
    D, P = POINTER(eqat_desc), c_void_p
    sigs = {
        "eqat_status_string": (c_char_p, [c_int]),
        "eqat_version": (c_int, []),
        "eqat_workspace_bytes": (c_size_t, [D, c_int]),
        "eqat_device_status": (c_int, [POINTER(c_int), POINTER(c_int)]),
        "eqat_selftest_wait_expiry": (c_int, [c_int, P]),
        "eqat_minmax_init": (c_int, [D, P, P, P, P]),
        "eqat_fakequant_weight": (c_int, [D, P, P, P, P, P]),
        "qlinear_fakequant_fwd": (c_int, [D, P, P, P, P, P, P, P]),
        "eqat_ste_bwd": (c_int, [D, P, P, P, P, P, P, P, P]),
        "qlinear_fakequant_bwd": (c_int, [D, P, P, P, P, P, P, P, P, P, P, P, c_size_t, P]),
        "qlinear_fakequant_bwd_noalloc": (c_int, [D, P, P, P, P, P, P, P, P, P, P, P]),
        "eqat_quantize_pack": (c_int, [D, P, P, P, P, P, P, P]),
        "eqat_pack": (c_int, [D, P, P, P]),
        "eqat_unpack": (c_int, [D, P, P, P]),
        "eqat_pack_zeros": (c_int, [D, P, P, P]),
        "eqat_unpack_zeros": (c_int, [D, P, P, P]),
        "qlinear_packed_fwd": (c_int, [D, P, P, P, P, P, P]),
        "qlinear_packed_bwd_dx": (c_int, [D, P, P, P, P, P, P]),
        "qlinear_packed_bwd_ds": (c_int, [D, P, P, P, P, P, P, P, P, c_size_t, P]),
        "eqat_block_ap_step": (c_int, [POINTER(eqat_block_ap_linear), c_int, POINTER(c_int), P]),
        "eqat_e2e_qp_step": (c_int, [POINTER(eqat_e2e_qp_linear), c_int, POINTER(c_int), P]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


lib = _load()
LIB_PATH = _LIB_PATH


def status_string(status: int) -> str:
    return lib.eqat_status_string(int(status)).decode()


def make_desc(bits, group, out_features, in_features, tokens=0, dz_mode=0, zero_point_format=EQAT_ZP_U8) -> eqat_desc:
    return eqat_desc(int(bits), int(group), int(out_features), int(in_features), int(tokens), int(dz_mode),
                     int(zero_point_format))


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, where):
    if rc != EQAT_OK:
        raise EqatError(rc, where)


def workspace_bytes(desc, op) -> int:
    n = lib.eqat_workspace_bytes(ctypes.byref(desc), int(op))
    if n == ctypes.c_size_t(-1).value:
        raise EqatError(EQAT_ERR_SHAPE, "eqat_workspace_bytes")
    return int(n)


def device_status():
    st, det = c_int(0), c_int(0)
    _check(lib.eqat_device_status(ctypes.byref(st), ctypes.byref(det)), "eqat_device_status")
    return st.value, det.value


def eqat_selftest_wait_expiry(which):
    _check(lib.eqat_selftest_wait_expiry(int(which), _stream()), "eqat_selftest_wait_expiry")


def eqat_minmax_init(desc, W, s, z):
    _check(lib.eqat_minmax_init(ctypes.byref(desc), _ptr(W), _ptr(s), _ptr(z), _stream()), "eqat_minmax_init")


def eqat_fakequant_weight(desc, W, s, z, W_hat):
    _check(lib.eqat_fakequant_weight(ctypes.byref(desc), _ptr(W), _ptr(s), _ptr(z), _ptr(W_hat), _stream()),
           "eqat_fakequant_weight")


def qlinear_fakequant_fwd(desc, X, W, s, z, Y, W_hat):
    _check(lib.qlinear_fakequant_fwd(ctypes.byref(desc), _ptr(X), _ptr(W), _ptr(s), _ptr(z), _ptr(Y), _ptr(W_hat),
                                     _stream()), "qlinear_fakequant_fwd")


def eqat_ste_bwd(desc, dW_hat, W, s, z, dW, ds, dz):
    _check(lib.eqat_ste_bwd(ctypes.byref(desc), _ptr(dW_hat), _ptr(W), _ptr(s), _ptr(z), _ptr(dW), _ptr(ds), _ptr(dz),
                            _stream()), "eqat_ste_bwd")


def qlinear_fakequant_bwd(desc, X, dY, W, s, z, W_hat, dX, dW, ds, dz, workspace):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.qlinear_fakequant_bwd(ctypes.byref(desc), _ptr(X), _ptr(dY), _ptr(W), _ptr(s), _ptr(z), _ptr(W_hat),
                                     _ptr(dX), _ptr(dW), _ptr(ds), _ptr(dz), _ptr(workspace), nbytes, _stream()),
           "qlinear_fakequant_bwd")


NOALLOC_MAX_WEIGHT_ELEMS = 4 << 20


def qlinear_fakequant_bwd_noalloc(desc, X, dY, W, s, z, W_hat, dX, dW, ds, dz):
    """Block-AP backward without a caller-provided workspace: for callers that
    cannot allocate device memory (the scratch is a fixed 8 MiB array inside the
    library, so out*in <= NOALLOC_MAX_WEIGHT_ELEMS; calls on one device must not
    overlap; make the first call on a device outside any stream capture)."""
    _check(lib.qlinear_fakequant_bwd_noalloc(ctypes.byref(desc), _ptr(X), _ptr(dY), _ptr(W), _ptr(s), _ptr(z),
                                             _ptr(W_hat), _ptr(dX), _ptr(dW), _ptr(ds), _ptr(dz), _stream()),
           "qlinear_fakequant_bwd_noalloc")


def eqat_quantize_pack(desc, W, s, z, Wq_packed, z8, s16):
    _check(lib.eqat_quantize_pack(ctypes.byref(desc), _ptr(W), _ptr(s), _ptr(z), _ptr(Wq_packed), _ptr(z8), _ptr(s16),
                                  _stream()), "eqat_quantize_pack")


def eqat_pack(desc, codes, Wq_packed):
    _check(lib.eqat_pack(ctypes.byref(desc), _ptr(codes), _ptr(Wq_packed), _stream()), "eqat_pack")


def eqat_unpack(desc, Wq_packed, codes):
    _check(lib.eqat_unpack(ctypes.byref(desc), _ptr(Wq_packed), _ptr(codes), _stream()), "eqat_unpack")


def eqat_pack_zeros(desc, z8, z_packed):
    _check(lib.eqat_pack_zeros(ctypes.byref(desc), _ptr(z8), _ptr(z_packed), _stream()), "eqat_pack_zeros")


def eqat_unpack_zeros(desc, z_packed, z8):
    _check(lib.eqat_unpack_zeros(ctypes.byref(desc), _ptr(z_packed), _ptr(z8), _stream()), "eqat_unpack_zeros")


def qlinear_packed_fwd(desc, X, Wq_packed, s16, z8, Y):
    _check(lib.qlinear_packed_fwd(ctypes.byref(desc), _ptr(X), _ptr(Wq_packed), _ptr(s16), _ptr(z8), _ptr(Y),
                                  _stream()), "qlinear_packed_fwd")


def qlinear_packed_bwd_dx(desc, dY, Wq_packed, s16, z8, dX):
    _check(lib.qlinear_packed_bwd_dx(ctypes.byref(desc), _ptr(dY), _ptr(Wq_packed), _ptr(s16), _ptr(z8), _ptr(dX),
                                     _stream()), "qlinear_packed_bwd_dx")


def qlinear_packed_bwd_ds(desc, X, dY, Wq_packed, z8, s16, ds, dz=None, workspace=None):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.qlinear_packed_bwd_ds(ctypes.byref(desc), _ptr(X), _ptr(dY), _ptr(Wq_packed), _ptr(z8), _ptr(s16),
                                     _ptr(ds), _ptr(dz), _ptr(workspace), nbytes, _stream()),
           "qlinear_packed_bwd_ds")


def _addr(t):
    p = _ptr(t)
    return None if p is None else p.value


def _nbytes(t):
    return 0 if t is None else t.numel() * t.element_size()


def _run_block(fn, struct, rows, where):
    arr = (struct * len(rows))(*rows)
    failed = c_int(-1)
    rc = fn(arr, len(rows), ctypes.byref(failed), _stream())
    if rc != EQAT_OK:
        raise EqatError(rc, f"{where} (linear {failed.value})")


def eqat_block_ap_step(linears):
    """Block-AP forward + backward of every linear of a block in one call.  `linears`: dicts with desc, X, dY, W,
    s, z, Y, W_hat (or None), dX, dW, ds, dz (or None), workspace (or None)."""
    rows = [eqat_block_ap_linear(L["desc"], _addr(L["X"]), _addr(L["dY"]), _addr(L["W"]), _addr(L["s"]), _addr(L["z"]),
                                 _addr(L["Y"]), _addr(L.get("W_hat")), _addr(L["dX"]), _addr(L["dW"]), _addr(L["ds"]),
                                 _addr(L.get("dz")), _addr(L.get("workspace")), _nbytes(L.get("workspace")))
            for L in linears]
    _run_block(lib.eqat_block_ap_step, eqat_block_ap_linear, rows, "eqat_block_ap_step")


def eqat_e2e_qp_step(linears):
    """E2E-QP forward, dX and ds (dz) of every linear of a block in one call.  `linears`: dicts with desc, X, dY,
    Wq_packed, s16, z, Y, dX, ds, dz (or None), workspace (or None)."""
    rows = [eqat_e2e_qp_linear(L["desc"], _addr(L["X"]), _addr(L["dY"]), _addr(L["Wq_packed"]), _addr(L["s16"]),
                               _addr(L["z"]), _addr(L["Y"]), _addr(L["dX"]), _addr(L["ds"]), _addr(L.get("dz")),
                               _addr(L.get("workspace")), _nbytes(L.get("workspace")))
            for L in linears]
    _run_block(lib.eqat_e2e_qp_step, eqat_e2e_qp_linear, rows, "eqat_e2e_qp_step")
