"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and this package never imports the
CUDA library or its binding.

`build()` compiles `patconv_ref.c` and `blockgemm_ref.c` with gcc into
`libpatconv_ref.so` next to them; `conv()` runs one pattern-pruned layer,
`block_gemm()` one block-pruned matrix product, `depthwise()` one
pattern-pruned depthwise layer.  Floating-point inputs (fp32 or fp16 arrays) are
widened to double exactly before the call, so the oracle's result is the
double-precision value of the layer on the stored inputs.  Parity status:
pinned (see the header of patconv_ref.c).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "patconv_ref.c")
_SRC_GEMM = os.path.join(_HERE, "blockgemm_ref.c")
_LIB = os.path.join(_HERE, "libpatconv_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or stale."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_GEMM))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, _SRC_GEMM, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        I = ctypes.c_int
        lib.patconv_ref_f64.argtypes = [P, P, P, P, I, P, I, I, I, I, I, I, I, P, P]
        lib.patconv_ref_f64.restype = I
        lib.patconv_ref_i64.argtypes = [P, P, P, P, I, P, I, I, I, I, I, I, I, P]
        lib.patconv_ref_i64.restype = I
        lib.patconv_ref_threads.restype = I
        lib.patconv_ref_fused_f64.argtypes = [P, P, I, I, I, I, I, I, P]
        lib.patconv_ref_fused_f64.restype = I
        lib.patconv_ref_fused_i64.argtypes = [P, P, I, I, I, I, I, I, P, I, P, P]
        lib.patconv_ref_fused_i64.restype = I
        lib.blockgemm_ref_f64.argtypes = [P, P, P, P, P, I, ctypes.c_long, I, I, I, I, P, P]
        lib.blockgemm_ref_f64.restype = I
        lib.dwconv_ref_f64.argtypes = [P, P, P, P, I, P, I, I, I, I, I, I, P, P]
        lib.dwconv_ref_f64.restype = I
        _lib = lib
    return _lib


def threads() -> int:
    """Host threads the oracle uses (OpenMP's maximum)."""
    return int(_load().patconv_ref_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def out_shape(h: int, w: int, stride: int):
    return (h + 2 - 3) // stride + 1, (w + 2 - 3) // stride + 1


def conv(x, w, pid, masks, bias=None, relu=False, stride=1, with_scale=False):
    """One pattern-pruned 3x3 layer, padding 1.

    x     [N,H,W,Cin]   float16/32/64, or uint8 for the integer layer
    w     [Cout,Cin,3,3] same family as x (int8 for the integer layer); dense:
          values at pruned positions are ignored
    pid   [Cout,Cin] int16 pattern id per kernel, -1 = kernel removed
    masks [P] uint16, bit 3*dy+dx = tap kept
    bias  [Cout] float (int32 for the integer layer) or None
    Returns y [N,Ho,Wo,Cout] as float64 (int64 for the integer layer); with
    `with_scale` also S = |bias| + sum |w*x| per output (floating point only).
    """
    lib = _load()
    x = np.asarray(x)
    w = np.asarray(w)
    n, h, wd, c_in = x.shape
    c_out = w.shape[0]
    if w.shape != (c_out, c_in, 3, 3):
        raise ValueError("w must be [Cout,Cin,3,3]")
    pid = np.ascontiguousarray(pid, dtype=np.int16)
    masks = np.ascontiguousarray(masks, dtype=np.uint16)
    if pid.shape != (c_out, c_in):
        raise ValueError("pid must be [Cout,Cin]")
    ho, wo = out_shape(h, wd, stride)
    if x.dtype == np.uint8:
        if w.dtype != np.int8:
            raise ValueError("integer layer wants int8 weights")
        xc = np.ascontiguousarray(x)
        wc = np.ascontiguousarray(w)
        bc = None if bias is None else np.ascontiguousarray(bias, dtype=np.int32)
        y = np.empty((n, ho, wo, c_out), dtype=np.int64)
        rc = lib.patconv_ref_i64(_ptr(xc), _ptr(wc), _ptr(pid), _ptr(masks), len(masks), _ptr(bc),
                                 int(bool(relu)), n, h, wd, c_in, c_out, stride, _ptr(y))
        if rc:
            raise ValueError("oracle error %d" % rc)
        return y
    xc = np.ascontiguousarray(x, dtype=np.float64)
    wc = np.ascontiguousarray(w, dtype=np.float64)
    bc = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    y = np.empty((n, ho, wo, c_out), dtype=np.float64)
    s = np.empty_like(y) if with_scale else None
    rc = lib.patconv_ref_f64(_ptr(xc), _ptr(wc), _ptr(pid), _ptr(masks), len(masks), _ptr(bc),
                             int(bool(relu)), n, h, wd, c_in, c_out, stride, _ptr(y), _ptr(s))
    if rc:
        raise ValueError("oracle error %d" % rc)
    return (y, s) if with_scale else y


def conv_fused(x, w, pid, masks, bias=None, relu=False, stride=1, residual=None, pool=0,
               requant_scale=None, zero_point=0):
    """The layer followed by the operators fused behind it (paper Sec. 2.2): an optional
    element-wise addition of `residual` (shaped like the convolution's output), the optional
    ReLU, an optional 2x2 max-pool of stride 2 and, for the integer layer, an optional
    re-quantisation to uint8 with one fp32 scale per output channel.  The convolution is
    `conv` (its own pins apply); the operators behind it are plain loops in patconv_ref.c.
    Returns float64 (int64; uint8 when re-quantised)."""
    lib = _load()
    pre = conv(x, w, pid, masks, bias=bias, relu=False, stride=stride)
    n, ho, wo, c = pre.shape
    step = 2 if pool == 2 else 1
    if pool not in (0, 2):
        raise ValueError("pool must be 0 or 2")
    oshape = (n, ho // step, wo // step, c)
    if pre.dtype == np.int64:
        rc_ = None if residual is None else np.ascontiguousarray(residual, dtype=np.int32)
        if rc_ is not None and rc_.shape != pre.shape:
            raise ValueError("residual must be shaped like the convolution's output")
        sc = None if requant_scale is None else np.ascontiguousarray(requant_scale, dtype=np.float32)
        out_i = np.empty(oshape, dtype=np.int64) if sc is None else None
        out_u = np.empty(oshape, dtype=np.uint8) if sc is not None else None
        rc = lib.patconv_ref_fused_i64(_ptr(pre), _ptr(rc_), int(bool(relu)), int(pool), n, ho, wo, c,
                                       _ptr(sc), int(zero_point), _ptr(out_i), _ptr(out_u))
        if rc:
            raise ValueError("oracle error %d" % rc)
        return out_i if sc is None else out_u
    if requant_scale is not None:
        raise ValueError("re-quantisation belongs to the integer layer")
    rc_ = None if residual is None else np.ascontiguousarray(residual, dtype=np.float64)
    if rc_ is not None and rc_.shape != pre.shape:
        raise ValueError("residual must be shaped like the convolution's output")
    out = np.empty(oshape, dtype=np.float64)
    rc = lib.patconv_ref_fused_f64(_ptr(pre), _ptr(rc_), int(bool(relu)), int(pool), n, ho, wo, c, _ptr(out))
    if rc:
        raise ValueError("oracle error %d" % rc)
    return out


def block_gemm(x, w, row_keep, col_keep, br, bc, bias=None, relu=False, with_scale=False):
    """One block-pruned matrix product (paper Sec. 2.1, "Block-Based Pruning").

    x        [M,K]    float16/32/64: one row per pixel (NHWC) or token
    w        [Cout,K] dense; values at pruned positions are ignored
    row_keep [ceil(Cout/br), ceil(K/bc), br] uint8, 0 = this row of the block is pruned
    col_keep [ceil(Cout/br), ceil(K/bc), bc] uint8, 0 = this column of the block is pruned
    bias     [Cout] or None
    Returns y [M,Cout] float64; with `with_scale` also S = |bias| + sum |w*x| per output.
    """
    lib = _load()
    x = np.asarray(x)
    w = np.asarray(w)
    m, k = x.shape
    c_out = w.shape[0]
    if w.shape != (c_out, k):
        raise ValueError("w must be [Cout,K]")
    nbr, nbc = (c_out + br - 1) // br, (k + bc - 1) // bc
    rk = np.ascontiguousarray(row_keep, dtype=np.uint8)
    ck = np.ascontiguousarray(col_keep, dtype=np.uint8)
    if rk.shape != (nbr, nbc, br) or ck.shape != (nbr, nbc, bc):
        raise ValueError("row_keep / col_keep must be [blocks of rows, blocks of columns, br | bc]")
    xc = np.ascontiguousarray(x, dtype=np.float64)
    wc = np.ascontiguousarray(w, dtype=np.float64)
    bcst = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    y = np.empty((m, c_out), dtype=np.float64)
    s = np.empty_like(y) if with_scale else None
    rc = lib.blockgemm_ref_f64(_ptr(xc), _ptr(wc), _ptr(rk), _ptr(ck), _ptr(bcst), int(bool(relu)),
                               m, k, c_out, br, bc, _ptr(y), _ptr(s))
    if rc:
        raise ValueError("oracle error %d" % rc)
    return (y, s) if with_scale else y


def depthwise(x, w, pid, masks, bias=None, relu=False, stride=1, with_scale=False):
    """One depthwise pattern-pruned 3x3 layer, padding 1: every channel has one 3x3 kernel.

    x     [N,H,W,C] float16/32/64
    w     [C,3,3]   dense; values at pruned taps are ignored
    pid   [C] int16 pattern id per channel, -1 = the channel's kernel is removed
    masks [P] uint16, bit 3*dy+dx = tap kept
    Returns y [N,Ho,Wo,C] float64; with `with_scale` also S = |bias| + sum |w*x|.
    """
    lib = _load()
    x = np.asarray(x)
    n, h, wd, c = x.shape
    w = np.asarray(w)
    if w.shape != (c, 3, 3):
        raise ValueError("w must be [C,3,3]")
    pid = np.ascontiguousarray(pid, dtype=np.int16)
    if pid.shape != (c,):
        raise ValueError("pid must be [C]")
    masks = np.ascontiguousarray(masks, dtype=np.uint16)
    ho, wo = out_shape(h, wd, stride)
    xc = np.ascontiguousarray(x, dtype=np.float64)
    wc = np.ascontiguousarray(w, dtype=np.float64)
    bc = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    y = np.empty((n, ho, wo, c), dtype=np.float64)
    s = np.empty_like(y) if with_scale else None
    rc = lib.dwconv_ref_f64(_ptr(xc), _ptr(wc), _ptr(pid), _ptr(masks), len(masks), _ptr(bc),
                            int(bool(relu)), n, h, wd, c, stride, _ptr(y), _ptr(s))
    if rc:
        raise ValueError("oracle error %d" % rc)
    return (y, s) if with_scale else y
