"""ctypes binding of libpeqa_b200.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/peqa.h)
minus the ``peqa_`` prefix.  torch provides device memory and the current
stream; all arithmetic runs in the library's CUDA kernels.  There is no CPU
fallback: a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpeqa_b200.so")
_lib = None

OP_FWD, OP_BWD, OP_DECODE, OP_BWD_DS_FROM_Y, OP_BWD_DSDZ = 0, 1, 2, 3, 4

STATUS_NAMES = {
    0: "PEQA_OK", -1: "PEQA_ERR_NULL", -2: "PEQA_ERR_BAD_BITS", -3: "PEQA_ERR_BAD_SHAPE",
    -4: "PEQA_ERR_ALIGNMENT", -5: "PEQA_ERR_WORKSPACE", -6: "PEQA_ERR_ARCH", -7: "PEQA_ERR_CUDA",
    -8: "PEQA_ERR_DEVICE_TIMEOUT", -9: "PEQA_ERR_TOO_LARGE",
}


class PeqaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        extra = ""
        if status == -7 and _lib is not None:
            extra = f" (cudaError {_lib.peqa_last_cuda_error()})"
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}{extra}")


class _QWeight(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int32), ("out_features", ctypes.c_int32),
                ("in_features", ctypes.c_int32), ("group_size", ctypes.c_int32),
                ("qweight", ctypes.c_void_p), ("zeros", ctypes.c_void_p),
                ("scales", ctypes.c_void_p)]


class _LayerLinear(ctypes.Structure):
    _fields_ = [("w", _QWeight), ("X", ctypes.c_void_p), ("dY", ctypes.c_void_p), ("Y", ctypes.c_void_p),
                ("dX", ctypes.c_void_p), ("dS", ctypes.c_void_p), ("m", ctypes.c_void_p),
                ("v", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


class _LayerHostLinear(ctypes.Structure):
    _fields_ = [("w", _QWeight), ("h_X", ctypes.c_void_p), ("h_dY", ctypes.c_void_p), ("h_Y", ctypes.c_void_p),
                ("h_dX", ctypes.c_void_p), ("h_dS", ctypes.c_void_p), ("d_X", ctypes.c_void_p),
                ("d_dY", ctypes.c_void_p), ("d_Y", ctypes.c_void_p), ("d_dX", ctypes.c_void_p),
                ("d_dS", ctypes.c_void_p), ("d_m", ctypes.c_void_p), ("d_v", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


def lib() -> ctypes.CDLL:
    """Load the shared library (built by paper_2305_14152_b200.build); never falls back."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: run `python -m paper_2305_14152_b200.build` first; "
                "there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float,
                                 ctypes.c_size_t)
        qp = ctypes.POINTER(_QWeight)
        L.peqa_version.restype = ctypes.c_int
        L.peqa_last_cuda_error.restype = ctypes.c_int
        L.peqa_quantize_rtn.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp]
        L.peqa_quantize_search.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]
        L.peqa_quantize_search.restype = ctypes.c_int
        L.peqa_pack.argtypes = [vp, i32, i32, i32, vp, vp]
        L.peqa_unpack.argtypes = [vp, i32, i32, i32, vp, vp]
        L.peqa_workspace_bytes.argtypes = [i32, i32, qp]
        L.peqa_workspace_bytes.restype = sz
        L.peqa_qlinear_fwd.argtypes = [qp, vp, i32, vp, vp, sz, vp]
        L.peqa_qlinear_bwd.argtypes = [qp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.peqa_qlinear_decode.argtypes = [qp, vp, i32, vp, vp, sz, vp]
        L.peqa_scale_adamw.argtypes = [vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, i64, vp]
        L.peqa_train_step_host.argtypes = [qp, i32] + [vp] * 12 + [f32] * 5 + [i64, vp, sz, vp]
        L.peqa_check_status.argtypes = [vp]
        L.peqa_qlinear_decode_multitask.argtypes = [qp, vp, i32, vp, vp, i32, vp, vp]
        L.peqa_qlinear_decode_multitask.restype = ctypes.c_int
        L.peqa_qlinear_bwd_ds_adamw.argtypes = [qp, vp, vp, i32, vp, vp, vp, f32, f32, f32, f32, f32, i64, vp, sz, vp]
        L.peqa_qlinear_bwd_ds_adamw.restype = ctypes.c_int
        L.peqa_qlinear_bwd_dsdz.argtypes = [qp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.peqa_qlinear_bwd_dsdz.restype = ctypes.c_int
        L.peqa_qlinear_bwd_ds_from_y.argtypes = [qp, vp, vp, i32, vp, vp, sz, vp]
        L.peqa_qlinear_bwd_ds_from_y.restype = ctypes.c_int
        L.peqa_qlinear_bwd_ds_static.argtypes = [qp, vp, vp, i32, vp, vp]
        L.peqa_qlinear_bwd_ds_static.restype = ctypes.c_int
        L.peqa_bwd_ds_static_capacity_bytes.restype = sz
        L.peqa_decode_prepared_bytes.argtypes = [qp]
        L.peqa_decode_prepared_bytes.restype = sz
        L.peqa_decode_prepare.argtypes = [qp, vp, vp]
        L.peqa_decode_prepare.restype = ctypes.c_int
        L.peqa_decode_unprepare.argtypes = [qp, vp, vp, vp]
        L.peqa_decode_unprepare.restype = ctypes.c_int
        L.peqa_qlinear_decode_prepared.argtypes = [qp, vp, vp, i32, vp, vp, i32, vp, vp]
        L.peqa_qlinear_decode_prepared.restype = ctypes.c_int
        L.peqa_qlinear_fwd_zf.argtypes = [qp, vp, vp, i32, vp, vp]
        L.peqa_qlinear_fwd_zf.restype = ctypes.c_int
        L.peqa_qlinear_bwd_zf.argtypes = [qp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.peqa_qlinear_bwd_zf.restype = ctypes.c_int
        L.peqa_zero_adamw.argtypes = [vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, i64, vp]
        L.peqa_zero_adamw.restype = ctypes.c_int
        L.peqa_selftest_configure.argtypes = [i32, i32]
        L.peqa_selftest_configure.restype = ctypes.c_int
        L.peqa_layer_train_step.argtypes = [ctypes.POINTER(_LayerLinear), i32, i32, i32, f32, f32, f32, f32, f32,
                                            i64, vp]
        L.peqa_layer_train_step.restype = ctypes.c_int
        L.peqa_layer_train_step_host.argtypes = [ctypes.POINTER(_LayerHostLinear), i32, i32, f32, f32, f32, f32,
                                                 f32, i64, vp]
        L.peqa_layer_train_step_host.restype = ctypes.c_int
        L.peqa_probe_read.argtypes = [vp, sz, vp, sz, vp]
        L.peqa_probe_read.restype = ctypes.c_int
        for name in ("peqa_quantize_rtn", "peqa_pack", "peqa_unpack", "peqa_qlinear_fwd",
                     "peqa_qlinear_bwd", "peqa_qlinear_decode", "peqa_scale_adamw",
                     "peqa_train_step_host", "peqa_check_status"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise PeqaError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


@dataclass
class QWeight:
    """Device tensors of one PEQA layer: packed Q (int32 bit patterns), z (uint8), s (fp32)."""
    bits: int
    N: int
    K: int
    group_size: int          # 0 = per-channel
    qweight: torch.Tensor    # int32 [N, K*bits/32]
    zeros: torch.Tensor      # uint8 [N, G]
    scales: torch.Tensor     # float32 [N, G]

    @property
    def G(self) -> int:
        return 1 if self.group_size in (0, self.K) else self.K // self.group_size

    def c_struct(self) -> _QWeight:
        return _QWeight(self.bits, self.N, self.K, self.group_size, self.qweight.data_ptr(),
                        self.zeros.data_ptr(), self.scales.data_ptr())


def version() -> int:
    return lib().peqa_version()


def quantize_rtn(W: torch.Tensor, bits: int, group_size: int = 0, out: QWeight | None = None) -> QWeight:
    """Quantize W; with ``out`` the results are written into its existing tensors."""
    _dev(W, torch.float32, "W")
    N, K = W.shape
    if out is not None:
        q, z, s = out.qweight, out.zeros, out.scales
    else:
        G = 1 if group_size in (0, K) else max(K // max(group_size, 1), 1)
        words = max(K * bits // 32, 1)
        q = torch.empty((N, words), dtype=torch.int32, device=W.device)
        z = torch.empty((N, G), dtype=torch.uint8, device=W.device)
        s = torch.empty((N, G), dtype=torch.float32, device=W.device)
    _check(lib().peqa_quantize_rtn(W.data_ptr(), N, K, bits, group_size, q.data_ptr(), z.data_ptr(),
                                   s.data_ptr(), _stream()), "peqa_quantize_rtn")
    return out if out is not None else QWeight(bits, N, K, group_size, q, z, s)


def quantize_search(W: torch.Tensor, bits: int, group_size: int = 0, n_candidates: int = 32):
    """Quantize W with the clipping range searched per group; returns (QWeight, chosen u8 [N,G])."""
    _dev(W, torch.float32, "W")
    N, K = W.shape
    G = 1 if group_size in (0, K) else max(K // max(group_size, 1), 1)
    q = torch.empty((N, max(K * bits // 32, 1)), dtype=torch.int32, device=W.device)
    z = torch.empty((N, G), dtype=torch.uint8, device=W.device)
    s = torch.empty((N, G), dtype=torch.float32, device=W.device)
    chosen = torch.empty((N, G), dtype=torch.uint8, device=W.device)
    _check(lib().peqa_quantize_search(W.data_ptr(), N, K, bits, group_size, n_candidates, q.data_ptr(),
                                      z.data_ptr(), s.data_ptr(), chosen.data_ptr(), _stream()),
           "peqa_quantize_search")
    return QWeight(bits, N, K, group_size, q, z, s), chosen


def pack(codes: torch.Tensor, bits: int) -> torch.Tensor:
    _dev(codes, torch.uint8, "codes")
    N, K = codes.shape
    q = torch.empty((N, max(K * bits // 32, 1)), dtype=torch.int32, device=codes.device)
    _check(lib().peqa_pack(codes.data_ptr(), N, K, bits, q.data_ptr(), _stream()), "peqa_pack")
    return q


def unpack(qweight: torch.Tensor, K: int, bits: int) -> torch.Tensor:
    _dev(qweight, torch.int32, "qweight")
    N = qweight.shape[0]
    codes = torch.empty((N, K), dtype=torch.uint8, device=qweight.device)
    _check(lib().peqa_unpack(qweight.data_ptr(), N, K, bits, codes.data_ptr(), _stream()),
           "peqa_unpack")
    return codes


def workspace_bytes(op: int, T: int, w: QWeight) -> int:
    cs = w.c_struct()
    return int(lib().peqa_workspace_bytes(op, T, ctypes.byref(cs)))


def alloc_workspace(op: int, T: int, w: QWeight):
    n = workspace_bytes(op, T, w)
    if n == 0:
        return None
    return torch.empty(n, dtype=torch.uint8, device=w.qweight.device)


def _ws(ws):
    return (0, 0) if ws is None else (ws.data_ptr(), ws.numel() * ws.element_size())


def qlinear_fwd(w: QWeight, X: torch.Tensor, Y: torch.Tensor | None = None, workspace=None):
    _dev(X, torch.bfloat16, "X")
    T = X.shape[0]
    if Y is None:
        Y = torch.empty((T, w.N), dtype=torch.bfloat16, device=X.device)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_fwd(ctypes.byref(cs), X.data_ptr(), T, Y.data_ptr(), wp, wb,
                                  _stream()), "peqa_qlinear_fwd")
    return Y


def qlinear_bwd(w: QWeight, X, dY: torch.Tensor, dX=None, dS=None, workspace=None,
                need_dx: bool = True, need_ds: bool = True):
    _dev(dY, torch.bfloat16, "dY")
    T = dY.shape[0]
    if need_dx and dX is None:
        dX = torch.empty((T, w.K), dtype=torch.bfloat16, device=dY.device)
    if need_ds and dS is None:
        dS = torch.empty((w.N, w.G), dtype=torch.float32, device=dY.device)
    if need_ds and workspace is None:
        workspace = alloc_workspace(OP_BWD, T, w)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_bwd(ctypes.byref(cs), _ptr(X), dY.data_ptr(), T,
                                  _ptr(dX) if need_dx else 0, _ptr(dS) if need_ds else 0,
                                  wp, wb, _stream()), "peqa_qlinear_bwd")
    return dX, dS


def qlinear_decode(w: QWeight, X: torch.Tensor, Y: torch.Tensor | None = None, workspace=None):
    _dev(X, torch.bfloat16, "X")
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(OP_DECODE, M, w)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_decode(ctypes.byref(cs), X.data_ptr(), M, Y.data_ptr(), wp, wb,
                                     _stream()), "peqa_qlinear_decode")
    return Y


def scale_adamw(scales, dS, m, v, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1):
    for t, n in ((scales, "scales"), (dS, "dS"), (m, "m"), (v, "v")):
        _dev(t, torch.float32, n)
    _check(lib().peqa_scale_adamw(scales.data_ptr(), dS.data_ptr(), m.data_ptr(), v.data_ptr(),
                                  scales.numel(), lr, beta1, beta2, eps, weight_decay, step,
                                  _stream()), "peqa_scale_adamw")


def train_step_host(w: QWeight, h_X, h_dY, h_Y, h_dX, h_dS, d_X, d_dY, d_Y, d_dX, d_dS, d_m, d_v,
                    lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1,
                    workspace=None):
    """Host-buffer training step: h_* are CPU tensors (pinned preferred), d_* device staging."""
    T = h_X.shape[0]
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_train_step_host(
        ctypes.byref(cs), T, h_X.data_ptr(), h_dY.data_ptr(), h_Y.data_ptr(), h_dX.data_ptr(),
        h_dS.data_ptr(), d_X.data_ptr(), d_dY.data_ptr(), d_Y.data_ptr(), d_dX.data_ptr(),
        d_dS.data_ptr(), d_m.data_ptr(), d_v.data_ptr(), lr, beta1, beta2, eps, weight_decay, step,
        wp, wb, _stream()), "peqa_train_step_host")


def qlinear_decode_multitask(w: QWeight, scale_table: torch.Tensor, task_ids: torch.Tensor,
                             X: torch.Tensor, Y=None):
    """Decode with one scale vector per task: scale_table fp32 [n_tasks, N], task_ids int32 [M]."""
    _dev(X, torch.bfloat16, "X")
    _dev(scale_table, torch.float32, "scale_table")
    _dev(task_ids, torch.int32, "task_ids")
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=X.device)
    cs = w.c_struct()
    _check(lib().peqa_qlinear_decode_multitask(ctypes.byref(cs), scale_table.data_ptr(),
                                               scale_table.shape[0], task_ids.data_ptr(),
                                               X.data_ptr(), M, Y.data_ptr(), _stream()),
           "peqa_qlinear_decode_multitask")
    return Y


def qlinear_bwd_ds_adamw(w: QWeight, X: torch.Tensor, dY: torch.Tensor, m: torch.Tensor,
                         v: torch.Tensor, lr: float, beta1=0.9, beta2=0.999, eps=1e-8,
                         weight_decay=0.0, step=1, dS=None, workspace=None):
    """dS and the AdamW step on w.scales (in place) in one pass."""
    _dev(X, torch.bfloat16, "X")
    _dev(dY, torch.bfloat16, "dY")
    T = dY.shape[0]
    if dS is None:
        dS = torch.empty((w.N, w.G), dtype=torch.float32, device=dY.device)
    if workspace is None:
        workspace = alloc_workspace(OP_BWD, T, w)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_bwd_ds_adamw(ctypes.byref(cs), X.data_ptr(), dY.data_ptr(), T,
                                           dS.data_ptr(), m.data_ptr(), v.data_ptr(), lr, beta1,
                                           beta2, eps, weight_decay, step, wp, wb, _stream()),
           "peqa_qlinear_bwd_ds_adamw")
    return dS


@dataclass
class LayerLinear:
    """Buffers of one linear of a layer step (all device tensors; m, v may be None when the
    optimizer step is not applied; workspace may be None when the layer needs none)."""
    w: QWeight
    X: torch.Tensor          # bf16 [T, K]
    dY: torch.Tensor         # bf16 [T, N]
    Y: torch.Tensor          # bf16 [T, N] out
    dX: torch.Tensor         # bf16 [T, K] out
    dS: torch.Tensor         # fp32 [N, G] out
    m: torch.Tensor | None = None
    v: torch.Tensor | None = None
    workspace: torch.Tensor | None = None


def layer_train_step(linears, lr: float = 0.0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1,
                     apply_adamw=True) -> None:
    """Forward, dX and dS (and, with apply_adamw, the AdamW step on the scales) of every linear of
    `linears` in one library call."""
    arr = (_LayerLinear * len(linears))()
    T = linears[0].dY.shape[0]
    for a, L in zip(arr, linears):
        _dev(L.X, torch.bfloat16, "X")
        _dev(L.dY, torch.bfloat16, "dY")
        _dev(L.Y, torch.bfloat16, "Y")
        _dev(L.dX, torch.bfloat16, "dX")
        _dev(L.dS, torch.float32, "dS")
        if L.dY.shape[0] != T or L.X.shape[0] != T:
            raise ValueError("all linears of a layer step take the same number of tokens")
        wp, wb = _ws(L.workspace)
        a.w = L.w.c_struct()
        a.X, a.dY, a.Y, a.dX, a.dS = (L.X.data_ptr(), L.dY.data_ptr(), L.Y.data_ptr(), L.dX.data_ptr(),
                                      L.dS.data_ptr())
        a.m, a.v = _ptr(L.m), _ptr(L.v)
        a.workspace, a.workspace_bytes = wp, wb
    _check(lib().peqa_layer_train_step(arr, len(linears), T, 1 if apply_adamw else 0, lr, beta1, beta2, eps,
                                       weight_decay, step, _stream()), "peqa_layer_train_step")


@dataclass
class HostLinear:
    """Buffers of one linear of a host-buffer layer step: h_* are CPU tensors (pinned for the copies
    to overlap), d_* device staging of the same shapes, not shared with another linear of the call."""
    w: QWeight
    h_X: torch.Tensor        # bf16 [T, K] in
    h_dY: torch.Tensor       # bf16 [T, N] in
    h_Y: torch.Tensor        # bf16 [T, N] out
    h_dX: torch.Tensor       # bf16 [T, K] out
    h_dS: torch.Tensor       # fp32 [N, G] out
    d_X: torch.Tensor
    d_dY: torch.Tensor
    d_Y: torch.Tensor
    d_dX: torch.Tensor
    d_dS: torch.Tensor
    d_m: torch.Tensor
    d_v: torch.Tensor
    workspace: torch.Tensor | None = None


def layer_train_step_host(linears, lr: float, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1) -> None:
    """The host-buffer training step of every linear of `linears` in one library call; the copies of
    a linear overlap the kernels of its neighbours."""
    arr = (_LayerHostLinear * len(linears))()
    T = linears[0].h_X.shape[0]
    for a, L in zip(arr, linears):
        if L.h_X.shape[0] != T or L.h_dY.shape[0] != T:
            raise ValueError("all linears of a layer step take the same number of tokens")
        for t in (L.h_X, L.h_dY, L.h_Y, L.h_dX, L.h_dS):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("h_* must be contiguous CPU tensors")
        for t, dt, nm in ((L.d_X, torch.bfloat16, "d_X"), (L.d_dY, torch.bfloat16, "d_dY"),
                          (L.d_Y, torch.bfloat16, "d_Y"), (L.d_dX, torch.bfloat16, "d_dX"),
                          (L.d_dS, torch.float32, "d_dS"), (L.d_m, torch.float32, "d_m"),
                          (L.d_v, torch.float32, "d_v")):
            _dev(t, dt, nm)
        wp, wb = _ws(L.workspace)
        a.w = L.w.c_struct()
        a.h_X, a.h_dY, a.h_Y, a.h_dX, a.h_dS = (L.h_X.data_ptr(), L.h_dY.data_ptr(), L.h_Y.data_ptr(),
                                                L.h_dX.data_ptr(), L.h_dS.data_ptr())
        a.d_X, a.d_dY, a.d_Y, a.d_dX, a.d_dS = (L.d_X.data_ptr(), L.d_dY.data_ptr(), L.d_Y.data_ptr(),
                                                L.d_dX.data_ptr(), L.d_dS.data_ptr())
        a.d_m, a.d_v = L.d_m.data_ptr(), L.d_v.data_ptr()
        a.workspace, a.workspace_bytes = wp, wb
    _check(lib().peqa_layer_train_step_host(arr, len(linears), T, lr, beta1, beta2, eps, weight_decay, step,
                                            _stream()), "peqa_layer_train_step_host")


def qlinear_bwd_dsdz(w: QWeight, X: torch.Tensor, dY: torch.Tensor, dS=None, dZ=None, workspace=None):
    """Scale gradient and zero-point gradient from the same dW tiles."""
    _dev(X, torch.bfloat16, "X")
    _dev(dY, torch.bfloat16, "dY")
    T = dY.shape[0]
    if dS is None:
        dS = torch.empty((w.N, w.G), dtype=torch.float32, device=dY.device)
    if dZ is None:
        dZ = torch.empty((w.N, w.G), dtype=torch.float32, device=dY.device)
    if workspace is None:
        workspace = alloc_workspace(OP_BWD_DSDZ, T, w)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_bwd_dsdz(ctypes.byref(cs), X.data_ptr(), dY.data_ptr(), T,
                                       dS.data_ptr(), dZ.data_ptr(), wp, wb, _stream()),
           "peqa_qlinear_bwd_dsdz")
    return dS, dZ


def qlinear_bwd_ds_from_y(w: QWeight, dY: torch.Tensor, Y: torch.Tensor, dS=None, workspace=None):
    """Per-channel dS from the stored forward output: (sum_t dY*Y) / s."""
    _dev(dY, torch.bfloat16, "dY")
    _dev(Y, torch.bfloat16, "Y")
    T = dY.shape[0]
    if dS is None:
        dS = torch.empty((w.N, 1), dtype=torch.float32, device=dY.device)
    if workspace is None:
        workspace = alloc_workspace(OP_BWD_DS_FROM_Y, T, w)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_bwd_ds_from_y(ctypes.byref(cs), dY.data_ptr(), Y.data_ptr(), T,
                                            dS.data_ptr(), wp, wb, _stream()),
           "peqa_qlinear_bwd_ds_from_y")
    return dS


def qlinear_bwd_ds_static(w: QWeight, X: torch.Tensor, dY: torch.Tensor, dS: torch.Tensor):
    """dS through the library's built-in scratch array; the caller supplies only inputs and
    the output tensor, and nothing is allocated on the way."""
    _dev(X, torch.bfloat16, "X")
    _dev(dY, torch.bfloat16, "dY")
    _dev(dS, torch.float32, "dS")
    cs = w.c_struct()
    _check(lib().peqa_qlinear_bwd_ds_static(ctypes.byref(cs), X.data_ptr(), dY.data_ptr(),
                                            dY.shape[0], dS.data_ptr(), _stream()),
           "peqa_qlinear_bwd_ds_static")
    return dS


def bwd_ds_static_capacity_bytes() -> int:
    return int(lib().peqa_bwd_ds_static_capacity_bytes())


def decode_prepared_bytes(w: QWeight) -> int:
    cs = w.c_struct()
    return int(lib().peqa_decode_prepared_bytes(ctypes.byref(cs)))


def decode_prepared_supported(w: QWeight) -> bool:
    """True when qlinear_decode_prepared serves this layer: K % 128 == 0, N % 8 == 0 and one scale
    per channel, groups of 64, 128 or 256 columns, or groups that are multiples of 512 columns."""
    g = w.group_size or w.K
    return decode_prepared_bytes(w) > 0 and (g == w.K or g % 512 == 0 or g in (64, 128, 256))


def decode_prepare(w: QWeight) -> torch.Tensor:
    """Prepared copy of w.qweight for qlinear_decode_prepared (int32 bit patterns, flat)."""
    n = decode_prepared_bytes(w)
    if n == 0:
        raise PeqaError(-3, "peqa_decode_prepared_bytes")
    out = torch.empty(n // 4, dtype=torch.int32, device=w.qweight.device)
    cs = w.c_struct()
    _check(lib().peqa_decode_prepare(ctypes.byref(cs), out.data_ptr(), _stream()), "peqa_decode_prepare")
    return out


def decode_unprepare(w: QWeight, prepared: torch.Tensor, out=None) -> torch.Tensor:
    """Canonical packed matrix rebuilt from a prepared buffer."""
    _dev(prepared, torch.int32, "prepared")
    if out is None:
        out = torch.empty((w.N, w.K * w.bits // 32), dtype=torch.int32, device=prepared.device)
    _dev(out, torch.int32, "out")
    cs = w.c_struct()
    _check(lib().peqa_decode_unprepare(ctypes.byref(cs), prepared.data_ptr(), out.data_ptr(), _stream()),
           "peqa_decode_unprepare")
    return out


def qlinear_decode_prepared(w: QWeight, prepared: torch.Tensor, X: torch.Tensor, Y=None,
                            scale_table=None, task_ids=None):
    """Decode from the prepared weights; with scale_table [n_tasks, N, G] and task_ids [M] every
    token uses the scales of its own task."""
    _dev(prepared, torch.int32, "prepared")
    _dev(X, torch.bfloat16, "X")
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, w.N), dtype=torch.bfloat16, device=X.device)
    n_tasks = 0
    if task_ids is not None:
        _dev(scale_table, torch.float32, "scale_table")
        _dev(task_ids, torch.int32, "task_ids")
        n_tasks = scale_table.shape[0]
    cs = w.c_struct()
    _check(lib().peqa_qlinear_decode_prepared(ctypes.byref(cs), prepared.data_ptr(), X.data_ptr(), M,
                                              Y.data_ptr(), _ptr(scale_table), n_tasks, _ptr(task_ids),
                                              _stream()), "peqa_qlinear_decode_prepared")
    return Y


def probe_read(buf: torch.Tensor, sink: torch.Tensor) -> None:
    """Read-only pass over ``buf`` (measurement aid); sink: int32 device tensor, one word per SM."""
    _check(lib().peqa_probe_read(buf.data_ptr(), buf.numel() * buf.element_size(), sink.data_ptr(),
                                 sink.numel() * sink.element_size(), _stream()), "peqa_probe_read")


def qlinear_fwd_zf(w: QWeight, zeros_f: torch.Tensor, X: torch.Tensor, Y=None):
    """Forward with real-valued zero-points zeros_f fp32 [N, G] (App. K)."""
    _dev(zeros_f, torch.float32, "zeros_f")
    _dev(X, torch.bfloat16, "X")
    T = X.shape[0]
    if Y is None:
        Y = torch.empty((T, w.N), dtype=torch.bfloat16, device=X.device)
    cs = w.c_struct()
    _check(lib().peqa_qlinear_fwd_zf(ctypes.byref(cs), zeros_f.data_ptr(), X.data_ptr(), T, Y.data_ptr(),
                                     _stream()), "peqa_qlinear_fwd_zf")
    return Y


def qlinear_bwd_zf(w: QWeight, zeros_f: torch.Tensor, X, dY: torch.Tensor, need_dx=True, need_grads=True,
                   workspace=None):
    """dX and/or (dS, dZ) with real-valued zero-points; returns (dX, dS, dZ)."""
    _dev(zeros_f, torch.float32, "zeros_f")
    _dev(dY, torch.bfloat16, "dY")
    T = dY.shape[0]
    dX = torch.empty((T, w.K), dtype=torch.bfloat16, device=dY.device) if need_dx else None
    dS = torch.empty((w.N, w.G), dtype=torch.float32, device=dY.device) if need_grads else None
    dZ = torch.empty((w.N, w.G), dtype=torch.float32, device=dY.device) if need_grads else None
    if need_grads and workspace is None:
        workspace = alloc_workspace(OP_BWD_DSDZ, T, w)
    cs = w.c_struct()
    wp, wb = _ws(workspace)
    _check(lib().peqa_qlinear_bwd_zf(ctypes.byref(cs), zeros_f.data_ptr(), _ptr(X), dY.data_ptr(), T,
                                     _ptr(dX), _ptr(dS), _ptr(dZ), wp, wb, _stream()), "peqa_qlinear_bwd_zf")
    return dX, dS, dZ


def zero_adamw(zeros_f, dZ, m, v, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1):
    for t, n in ((zeros_f, "zeros_f"), (dZ, "dZ"), (m, "m"), (v, "v")):
        _dev(t, torch.float32, n)
    _check(lib().peqa_zero_adamw(zeros_f.data_ptr(), dZ.data_ptr(), m.data_ptr(), v.data_ptr(),
                                 zeros_f.numel(), lr, beta1, beta2, eps, weight_decay, step, _stream()),
           "peqa_zero_adamw")


def selftest_configure(wait_limit_us: int = 0, starve_forward: bool = False) -> None:
    """Test knob of the bounded waits; selftest_configure() restores the defaults."""
    _check(lib().peqa_selftest_configure(int(wait_limit_us), 1 if starve_forward else 0),
           "peqa_selftest_configure")


def check_status() -> None:
    _check(lib().peqa_check_status(_stream()), "peqa_check_status")
