"""PEQA reference oracle (CPU, fp64) -- test infrastructure only.

Thin numpy/ctypes front for ``peqa_oracle.c``.  Nothing in the CUDA package
imports this module and this module imports nothing from it.  Only tests, the
smoke check and the benchmark's CPU-baseline leg may use it.

Every function mirrors one operation of the paper (arXiv 2305.14152):
Eq. 1 (RTN quantization), the packed b-bit layout, the layer built on Eq. 2
(forward, dX, dS) and AdamW on the scales (App. A).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "peqa_oracle.c")
_LIB = os.path.join(_HERE, "libpeqa_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    lib = _load()
    lib.oracle_num_threads.restype = ctypes.c_int
    return int(lib.oracle_num_threads())


def _group(K: int, group_size: int) -> int:
    g = K if group_size in (0, K) else group_size
    if K % g != 0:
        raise ValueError("group size must divide K")
    return g


def quantize_rtn(W: np.ndarray, bits: int, group_size: int = 0):
    """Eq. 1 in binary32.  Returns (codes u8 [N,K], zeros u8 [N,G], scales f32 [N,G])."""
    W = _c(W, np.float32)
    N, K = W.shape
    g = _group(K, group_size)
    G = K // g
    codes = np.empty((N, K), np.uint8)
    zeros = np.empty((N, G), np.uint8)
    scales = np.empty((N, G), np.float32)
    _load().oracle_quantize_rtn(_p(W), N, K, bits, g, _p(codes), _p(zeros), _p(scales))
    return codes, zeros, scales


def quantize_rtn_f64(W: np.ndarray, bits: int, group_size: int = 0):
    """Eq. 1 with binary64 quotients; only for counting precision-dependent codes."""
    W = _c(W, np.float32)
    N, K = W.shape
    g = _group(K, group_size)
    G = K // g
    codes = np.empty((N, K), np.uint8)
    zeros = np.empty((N, G), np.uint8)
    scales = np.empty((N, G), np.float64)
    _load().oracle_quantize_rtn_f64(_p(W), N, K, bits, g, _p(codes), _p(zeros), _p(scales))
    return codes, zeros, scales


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    if K % 32:
        raise ValueError("K must be a multiple of 32")
    words = np.empty((N, K * bits // 32), np.uint32)
    _load().oracle_pack(_p(codes), N, K, bits, _p(words))
    return words


def unpack(words: np.ndarray, K: int, bits: int) -> np.ndarray:
    words = _c(words, np.uint32)
    N = words.shape[0]
    assert words.shape[1] == K * bits // 32
    codes = np.empty((N, K), np.uint8)
    _load().oracle_unpack(_p(words), N, K, bits, _p(codes))
    return codes


def _sel(sel):
    if sel is None:
        return None, 0, None
    a = _c(sel, np.int32)
    return a, int(a.size), _p(a)


def fwd(X_bits, qweight, zeros, scales, bits: int, group_size: int = 0, tokens=None) -> np.ndarray:
    """Y = X W_hat^T in fp64.  X_bits: bf16 bit patterns uint16 [T,K]; qweight packed."""
    X_bits = _c(X_bits, np.uint16)
    T, K = X_bits.shape
    g = _group(K, group_size)
    codes = unpack(qweight, K, bits)
    N = codes.shape[0]
    zeros = _c(zeros, np.uint8).reshape(N, K // g)
    scales = _c(scales, np.float32).reshape(N, K // g)
    keep, n_sel, ptr = _sel(tokens)
    rows = n_sel if tokens is not None else T
    Y = np.empty((rows, N), np.float64)
    _load().oracle_fwd(_p(X_bits), T, _p(codes), _p(zeros), _p(scales), N, K, g,
                       ptr, n_sel, _p(Y))
    return Y


def bwd_dx(dY_bits, qweight, zeros, scales, K: int, bits: int, group_size: int = 0,
           tokens=None) -> np.ndarray:
    """dX = dY W_hat in fp64.  dY_bits: bf16 bit patterns uint16 [T,N]."""
    dY_bits = _c(dY_bits, np.uint16)
    T, N = dY_bits.shape
    g = _group(K, group_size)
    codes = unpack(qweight, K, bits)
    assert codes.shape[0] == N
    zeros = _c(zeros, np.uint8).reshape(N, K // g)
    scales = _c(scales, np.float32).reshape(N, K // g)
    keep, n_sel, ptr = _sel(tokens)
    rows = n_sel if tokens is not None else T
    dX = np.empty((rows, K), np.float64)
    _load().oracle_bwd_dx(_p(dY_bits), T, _p(codes), _p(zeros), _p(scales), N, K, g,
                          ptr, n_sel, _p(dX))
    return dX


def bwd_ds(X_bits, dY_bits, qweight, zeros, bits: int, group_size: int = 0,
           rows=None) -> np.ndarray:
    """dS[i,g] = sum_{j in g} (Q-z)[i,j] (dY^T X)[i,j] in fp64."""
    X_bits = _c(X_bits, np.uint16)
    dY_bits = _c(dY_bits, np.uint16)
    T, K = X_bits.shape
    N = dY_bits.shape[1]
    assert dY_bits.shape[0] == T
    g = _group(K, group_size)
    codes = unpack(qweight, K, bits)
    assert codes.shape[0] == N
    zeros = _c(zeros, np.uint8).reshape(N, K // g)
    keep, n_sel, ptr = _sel(rows)
    nrows = n_sel if rows is not None else N
    dS = np.empty((nrows, K // g), np.float64)
    _load().oracle_bwd_ds(_p(X_bits), _p(dY_bits), T, _p(codes), _p(zeros), N, K, g,
                          ptr, n_sel, _p(dS))
    return dS


def fwd_multitask(X_bits, qweight, zeros, scale_table, task_ids, bits: int, group_size: int = 0) -> np.ndarray:
    """Forward in which token m uses the scales of task task_ids[m] (Sec. 3.3: Q and z are shared
    by all tasks, s is task-specific).  scale_table is [n_tasks, N] for one scale per channel or
    [n_tasks, N, G] for grouped scales (Sec. 4.2)."""
    X_bits = _c(X_bits, np.uint16)
    scale_table = _c(scale_table, np.float32)
    task_ids = np.asarray(task_ids, dtype=np.int64)
    n_tasks, N = scale_table.shape[:2]
    Y = np.empty((X_bits.shape[0], N), np.float64)
    for task in range(n_tasks):
        rows = np.nonzero(task_ids == task)[0]
        if rows.size:
            Y[rows] = fwd(X_bits[rows], qweight, zeros, scale_table[task].reshape(N, -1), bits, group_size)
    return Y


def bwd_dz(X_bits, dY_bits, scales, group_size: int = 0, rows=None) -> np.ndarray:
    """dZ[i,g] = -s[i,g] sum_{j in g} (dY^T X)[i,j] in fp64 (App. K: trainable zero-points)."""
    X_bits = _c(X_bits, np.uint16)
    dY_bits = _c(dY_bits, np.uint16)
    T, K = X_bits.shape
    N = dY_bits.shape[1]
    assert dY_bits.shape[0] == T
    g = _group(K, group_size)
    scales = _c(scales, np.float32).reshape(N, K // g)
    keep, n_sel, ptr = _sel(rows)
    nrows = n_sel if rows is not None else N
    dZ = np.empty((nrows, K // g), np.float64)
    _load().oracle_bwd_dz(_p(X_bits), _p(dY_bits), T, _p(scales), N, K, g, ptr, n_sel, _p(dZ))
    return dZ


def bwd_ds_from_y(dY_bits, Y_bits, scales) -> np.ndarray:
    """Per-channel dS[i] = (sum_t dY[t,i] Y[t,i]) / s[i] in fp64, from the stored bf16 output."""
    dY_bits = _c(dY_bits, np.uint16)
    Y_bits = _c(Y_bits, np.uint16)
    T, N = dY_bits.shape
    assert Y_bits.shape == (T, N)
    scales = _c(scales, np.float32).reshape(N)
    dS = np.empty((N, 1), np.float64)
    _load().oracle_bwd_ds_from_y(_p(dY_bits), _p(Y_bits), _p(scales), T, N, _p(dS))
    return dS


def adamw(s, grad, m, v, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, step=1):
    """One AdamW step on the scales, fp64 arithmetic on the fp32 state."""
    s = _c(s, np.float32).ravel()
    grad = _c(grad, np.float32).ravel()
    m = _c(m, np.float32).ravel()
    v = _c(v, np.float32).ravel()
    n = s.size
    so = np.empty(n, np.float64)
    mo = np.empty(n, np.float64)
    vo = np.empty(n, np.float64)
    lib = _load()
    lib.oracle_adamw.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int64] + [ctypes.c_double] * 5 + \
        [ctypes.c_int64] + [ctypes.c_void_p] * 3
    lib.oracle_adamw(_p(s), _p(grad), _p(m), _p(v), n, float(lr), float(beta1), float(beta2),
                     float(eps), float(weight_decay), int(step), _p(so), _p(mo), _p(vo))
    return so, mo, vo


def quantize_search(W: np.ndarray, bits: int, group_size: int = 0, n_cand: int = 32):
    """Eq. 1 with the clipping range searched per (row, group) for the smallest reconstruction
    error (Sec. 3.2's "initialized to minimize"; the search is this library's reading).
    Returns (codes, zeros, scales, chosen candidate u8 [N,G], error f64 [N,G])."""
    W = _c(W, np.float32)
    N, K = W.shape
    g = _group(K, group_size)
    G = K // g
    codes = np.empty((N, K), np.uint8)
    zeros = np.empty((N, G), np.uint8)
    scales = np.empty((N, G), np.float32)
    chosen = np.empty((N, G), np.uint8)
    err = np.empty((N, G), np.float64)
    _load().oracle_quantize_search(_p(W), N, K, bits, g, int(n_cand), _p(codes), _p(zeros), _p(scales),
                                   _p(chosen), _p(err))
    return codes, zeros, scales, chosen, err


def fwd_zf(X_bits, qweight, zeros_f, scales, bits: int, group_size: int = 0, tokens=None) -> np.ndarray:
    """Forward with a real-valued zero-point (App. K): Y = X (s*(Q - z))^T, z binary32 [N,G]."""
    X_bits = _c(X_bits, np.uint16)
    T, K = X_bits.shape
    g = _group(K, group_size)
    codes = unpack(qweight, K, bits)
    N = codes.shape[0]
    zeros_f = _c(zeros_f, np.float32).reshape(N, K // g)
    scales = _c(scales, np.float32).reshape(N, K // g)
    keep, n_sel, ptr = _sel(tokens)
    rows = n_sel if tokens is not None else T
    Y = np.empty((rows, N), np.float64)
    _load().oracle_fwd_zf(_p(X_bits), T, _p(codes), _p(zeros_f), _p(scales), N, K, g, ptr, n_sel, _p(Y))
    return Y


def bwd_dx_zf(dY_bits, qweight, zeros_f, scales, K: int, bits: int, group_size: int = 0, tokens=None) -> np.ndarray:
    dY_bits = _c(dY_bits, np.uint16)
    T, N = dY_bits.shape
    g = _group(K, group_size)
    codes = unpack(qweight, K, bits)
    zeros_f = _c(zeros_f, np.float32).reshape(N, K // g)
    scales = _c(scales, np.float32).reshape(N, K // g)
    keep, n_sel, ptr = _sel(tokens)
    rows = n_sel if tokens is not None else T
    dX = np.empty((rows, K), np.float64)
    _load().oracle_bwd_dx_zf(_p(dY_bits), T, _p(codes), _p(zeros_f), _p(scales), N, K, g, ptr, n_sel, _p(dX))
    return dX


def bwd_ds_zf(X_bits, dY_bits, qweight, zeros_f, bits: int, group_size: int = 0, rows=None) -> np.ndarray:
    X_bits = _c(X_bits, np.uint16)
    dY_bits = _c(dY_bits, np.uint16)
    T, K = X_bits.shape
    N = dY_bits.shape[1]
    g = _group(K, group_size)
    G = K // g
    codes = unpack(qweight, K, bits)
    zeros_f = _c(zeros_f, np.float32).reshape(N, G)
    keep, n_sel, ptr = _sel(rows)
    n_out = n_sel if rows is not None else N
    dS = np.empty((n_out, G), np.float64)
    _load().oracle_bwd_ds_zf(_p(X_bits), _p(dY_bits), T, _p(codes), _p(zeros_f), N, K, g, ptr, n_sel, _p(dS))
    return dS
